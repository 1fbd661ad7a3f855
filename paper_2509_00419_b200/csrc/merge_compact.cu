// lvlm_merge_compact: P_new = W_v x P_merged and P_compressed = [P_unmerged, P_new]
// (Section 3.2.1, paragraph 4), applied to the hidden states, to that layer's K and V and
// to the position ids.
//
// Launches: (1) a plan kernel, one CTA per sequence, turns `rank` into a source-row map for
// every output row, a destination for every input row and a merge weight for every image token;
// (2) one streaming kernel reads every input row of the hidden states once, moves it if it is
// kept and adds it to the weighted sum if it is merged; (3) one kernel compacts K and V in place.
#include "common.cuh"
#include "compact.cuh"
#include "merge.cuh"

namespace lvlm {

struct MergeLayout {
    int r1, r, Nout, V;
    HiddenGrid grid;
    size_t off_src, off_dst, off_wgt, off_meta, off_partial, total;
};

constexpr int kHidThreads = 256;       // streaming kernel: thread = 16-byte column group (+256, +512 ...)
constexpr int kHidMaxChunks = 4;       // column groups per thread: rows up to 4 * 256 * 8 = 8192 channels
constexpr int kNoRow = -2147483647 - 1;  // marks a slot of a row group that lies past the last row
constexpr int kHidCluster = 8;         // CTAs whose partial sums are added through shared memory

// One wave of CTAs over the whole batch (four per SM fit for rows up to 4096 channels, two beyond:
// the registers of the row groups in flight decide), at least 8 input rows each; clusters of 8.
HiddenGrid hidden_grid(const lvlm_dims* d) {
    HiddenGrid g;
    g.V = d->C / 8;
    const int per_sm = (g.V + kHidThreads - 1) / kHidThreads <= 2 ? 4 : 2;
    int cps = (per_sm * 148) / d->B;
    const int max_by_rows = (d->N + 7) / 8;
    cps = cps > max_by_rows ? max_by_rows : cps;
    cps = cps < 1 ? 1 : cps;
    g.cl = cps >= kHidCluster ? kHidCluster : 1;
    cps = cps / g.cl * g.cl;
    g.cps = cps;
    g.rpc = (d->N + cps - 1) / cps;
    return g;
}

static bool merge_layout(const lvlm_dims* d, MergeLayout* L) {
    if (!d || d->B <= 0 || d->N <= 0 || d->n <= 0 || d->C <= 0 || d->C % 8 || d->i0 < 0 ||
        d->k < 0 || d->k > d->n || (int64_t)d->i0 + d->n > d->N)
        return false;
    L->r1 = d->n - d->k;
    L->r = L->r1 > 0 ? L->r1 - 1 : 0;
    L->Nout = d->N - L->r;
    L->V = d->C / 8;
    L->grid = hidden_grid(d);
    const int cps = L->grid.cps;
    size_t off = 0;
    L->off_src = off;     off = align_up(off + (size_t)d->B * d->N * 4, 256);
    L->off_dst = off;     off = align_up(off + (size_t)d->B * d->N * 4, 256);
    L->off_wgt = off;     off = align_up(off + (size_t)d->B * d->n * 4, 256);
    L->off_meta = off;    off = align_up(off + (size_t)d->B * kMetaInts * 4, 256);
    L->off_partial = off; off = align_up(off + (size_t)d->B * (cps / L->grid.cl) * d->C * 4, 256);
    L->total = off;
    return true;
}

size_t merge_compact_workspace(const lvlm_dims* d) {
    if (d && d->merge_mode == LVLM_W_NEAREST_KEPT) return nearest_kept_workspace(d);
    MergeLayout L;
    return merge_layout(d, &L) ? L.total : 0;
}

__device__ __forceinline__ float block_sum_fixed(float v, float* scratch) {
    // fixed reduction tree: xor shuffles inside a warp, then warp 0 over the warp sums
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = (threadIdx.x < (blockDim.x >> 5)) ? scratch[threadIdx.x] : 0.f;
    if (threadIdx.x < 32) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
        if (threadIdx.x == 0) scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// Weight of the merged token at place p of the queue (p = 0 most important), normalised.
__device__ __forceinline__ float merge_weight(int mode, int p, int r1, float inv_sum,
                                              const float* __restrict__ w_custom) {
    switch (mode) {
        case LVLM_W_LINEAR_RANK: return (float)(r1 - p) * inv_sum;
        case LVLM_W_GEOMETRIC:   return ldexpf(1.0f, -(p < r1 - 1 ? p + 1 : r1 - 1));
        case LVLM_W_UNIFORM:     return inv_sum;
        default:                 return w_custom[p] * inv_sum;
    }
}

__device__ __forceinline__ uint32_t plan_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void plan_cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ int plan_ld_cluster(const int* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    int v;
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}

// A cluster of P CTAs per sequence (grid (P, B)): source map, destination map, weights, position ids,
// new length.  CTA r takes the r-th run of the image tokens: it counts its kept tokens, learns from the
// lower ranks how many came before, then writes the maps of its run (tile by tile, thread = token,
// coalesced).  The position ids are compacted in place in rounds of P x blockDim output rows: every CTA
// loads its rows of the round, a cluster barrier, then it stores them (a row's source lies at or behind it,
// so nothing a later round needs is overwritten).
__global__ void __launch_bounds__(1024)
merge_plan_kernel(const int32_t* __restrict__ rank, int32_t* pos_ids, int N, int i0, int n, int k,
                  int mode, float inv_sum, const float* __restrict__ w_custom,
                  int32_t* __restrict__ src_map, int32_t* __restrict__ dst_map,
                  float* __restrict__ wgt, int32_t* __restrict__ meta, int32_t* new_len,
                  int32_t* dev_status) {
    __shared__ int scan_scratch[33];
    __shared__ float fsum_scratch[33];
    __shared__ int s_total, s_first_drop, s_merged_tok;
    pdl_enter();
    const int b = blockIdx.y, P = (int)gridDim.x, cr = (int)plan_cluster_rank();
    const int r1 = n - k, r = r1 - 1, Nout = N - r;
    const int32_t* rk = rank + (int64_t)b * n;
    int32_t* src = src_map + (int64_t)b * N;
    int32_t* dst = dst_map + (int64_t)b * N;      // output row of every input row, -1 = merged away
    float* w = wgt + (int64_t)b * n;
    const int chunk = (n + P - 1) / P;
    const int c_lo = min(n, cr * chunk), c_hi = min(n, c_lo + chunk);
    if (threadIdx.x == 0) { s_total = 0; s_first_drop = n; s_merged_tok = -1; }

    if (mode == LVLM_W_CUSTOM) {
        float part = 0.f;
        for (int p = threadIdx.x; p < r1; p += blockDim.x) part += w_custom[p];
        const float tot = block_sum_fixed(part, fsum_scratch);
        inv_sum = 1.0f / tot;
    }
    __syncthreads();

    // kept tokens of my run
    bool bad = false;
    int mine = 0;
    for (int t0 = c_lo; t0 < c_hi; t0 += blockDim.x) {
        const int j = t0 + threadIdx.x;
        const int rj = j < c_hi ? rk[j] : n;
        if (j < c_hi && (rj < 0 || rj >= n)) bad = true;
        mine += j < c_hi && rj < k;
    }
    mine = warp_sum(mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&s_total, mine);
    plan_cluster_barrier();
    int kept_before = 0, kept_all = 0;
    for (int q = 0; q < P; ++q) {
        const int t = plan_ld_cluster(&s_total, q);
        kept_before += q < cr ? t : 0;
        kept_all += t;
    }
    if (kept_all != k) bad = true;

    // the maps of my run
    for (int t0 = c_lo; t0 < c_hi; t0 += blockDim.x) {
        const int j = t0 + threadIdx.x;
        const int rj = j < c_hi ? rk[j] : n;              // past the end: counts as dropped, writes nothing
        const int is_kept = j < c_hi && rj < k;
        int total;
        const int off = kept_before + block_exclusive_scan(is_kept, scan_scratch, &total);
        if (j < c_hi) {
            float wj = 0.f;
            if (is_kept) {
                if (off < k) src[i0 + off] = i0 + j;
                dst[i0 + j] = off < k ? i0 + off : -1;
            } else {
                dst[i0 + j] = -1;
                if (rj == k) s_merged_tok = j;
                int p = rj - k;
                p = p < 0 ? 0 : (p >= r1 ? r1 - 1 : p);
                wj = merge_weight(mode, p, r1, inv_sum, w_custom);
            }
            w[j] = wj;
        }
        int fd = (j < c_hi && !is_kept) ? j : n;           // first dropped token: one atomic per warp
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fd = min(fd, __shfl_xor_sync(0xFFFFFFFFu, fd, o));
        if ((threadIdx.x & 31) == 0 && fd < n) atomicMin(&s_first_drop, fd);
        kept_before += total;
    }
    // rows outside the image span, shared out over the CTAs
    for (int o = cr * blockDim.x + threadIdx.x; o < Nout; o += P * blockDim.x) {
        if (o < i0) { src[o] = o; dst[o] = o; }
        else if (o == i0 + k) src[o] = -1;
        else if (o > i0 + k) { src[o] = o + r; dst[o + r] = o; }
    }
    if (bad && dev_status) atomicOr(dev_status, LVLM_DEV_BOUNDS);
    plan_cluster_barrier();                               // the maps are complete, every CTA's findings are in place
    int first_drop = n, merged_tok = 0;
    for (int q = 0; q < P; ++q) {
        first_drop = min(first_drop, plan_ld_cluster(&s_first_drop, q));
        const int mt = plan_ld_cluster(&s_merged_tok, q);
        if (mt >= 0) merged_tok = mt;
    }
    if (cr == 0 && threadIdx.x == 0) {
        meta[b * kMetaInts + 0] = i0 + first_drop;       // first row whose content changes
        meta[b * kMetaInts + 1] = 0;                     // ticket counter of the merge blocks
        meta[b * kMetaInts + 2] = merged_tok;
        if (new_len) new_len[b] = Nout;
    }
    if (pos_ids) {
        int32_t* pid = pos_ids + (int64_t)b * N;
        const int pos_new = pid[i0 + merged_tok];         // read before any CTA stores (first store: after a barrier)
        for (int o0 = 0; o0 < Nout; o0 += P * blockDim.x) {
            const int o = o0 + cr * blockDim.x + threadIdx.x;
            int val = 0;
            if (o < Nout) { const int sidx = src[o]; val = sidx >= 0 ? pid[sidx] : pos_new; }
            plan_cluster_barrier();
            if (o < Nout) pid[o] = val;
        }
    }
    plan_cluster_barrier();                               // nobody leaves while its shared memory may still be read
}

__global__ void identity_len_kernel(int32_t* new_len, int B, int N) {
    pdl_enter();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) new_len[b] = N;
}

__device__ __forceinline__ uint32_t hid_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void hid_cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ int hid_ld_cluster_i32(const int* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    int v;
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}
__device__ __forceinline__ float4 hid_ld_cluster_f4(const float* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
    return v;
}

// Hidden states, out of place.  grid (CTAs per sequence, B), clusters of `cl` CTAs along x.  A CTA
// takes every grid.x-th group of two consecutive INPUT rows and reads each row exactly once: a kept
// row goes to its destination, a merged row is added, times its weight, to fp32 sums the thread
// keeps for its columns (its rows in increasing order).  The CTAs of a cluster add their sums in rank
// order through distributed shared memory and park one partial per cluster; the last cluster of
// the sequence to finish adds the partials in cluster order, rounds once to bf16 and writes P_new.
template <int CH>
__global__ void __launch_bounds__(kHidThreads, CH <= 2 ? 4 : 2)     // the occupancy hidden_grid() counts on
hidden_stream_kernel(const uint4* __restrict__ hidden, uint4* __restrict__ out,
                     int64_t hid_stride_b, int64_t out_stride_b,   // in uint4
                     int V, int N, int i0, int n, int k, int rpc, int cl,
                     const int32_t* __restrict__ dst_map, const float* __restrict__ wgt,
                     int32_t* meta, float* partial, uint4* __restrict__ scratch, int64_t scr_stride_b) {
    extern __shared__ __align__(16) float s_sum[];           // [V][8] this CTA's sums
    __shared__ int s_last;
    pdl_enter();
    const int b = blockIdx.y, cta = blockIdx.x, tid = threadIdx.x;
    const uint4* hin = hidden + (int64_t)b * hid_stride_b;
    uint4* hout = out + (int64_t)b * out_stride_b;
    const int32_t* dst = dst_map + (int64_t)b * N;
    const float* w = wgt ? wgt + (int64_t)b * n - i0 : nullptr;   // indexed by sequence position
    uint4* scr = scratch ? scratch + (int64_t)b * scr_stride_b : nullptr;
    const int i_hi = N;
    (void)rpc;

    float acc[CH][8];
#pragma unroll
    for (int ci = 0; ci < CH; ++ci)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[ci][e] = 0.f;

    // Groups of kG rows are dealt out round robin, so that every CTA gets the same mix of kept rows (read
    // and written) and merged rows (read only).  Two groups are in flight in turn: the loads of the next
    // one are issued before the current one is used.
    constexpr int kG = 2;
    auto load_group = [&](int ib, int* d, float* wj, uint4 (*x)[CH]) {
#pragma unroll
        for (int u = 0; u < kG; ++u) {
            const int i = ib + u;
            d[u] = i < i_hi ? dst[i] : kNoRow;
            wj[u] = (w && i < i_hi && i >= i0 && i < i0 + n) ? w[i] : 0.f;
#pragma unroll
            for (int ci = 0; ci < CH; ++ci) {
                const int c = tid + ci * kHidThreads;
                x[u][ci] = (i < i_hi && c < V) ? __ldg(hin + (int64_t)i * V + c) : make_uint4(0, 0, 0, 0);
            }
        }
    };
    auto use_group = [&](const int* d, const float* wj, const uint4 (*x)[CH]) {
#pragma unroll
        for (int u = 0; u < kG; ++u) {
            if (d[u] >= 0) {
#pragma unroll
                for (int ci = 0; ci < CH; ++ci) {
                    const int c = tid + ci * kHidThreads;
                    if (c < V) hout[(int64_t)d[u] * V + c] = x[u][ci];
                }
            } else if (d[u] <= -2 && d[u] != kNoRow) {        // a row set aside: scratch row -d-2
                if (scr) {
#pragma unroll
                    for (int ci = 0; ci < CH; ++ci) {
                        const int c = tid + ci * kHidThreads;
                        if (c < V) scr[(int64_t)(-d[u] - 2) * V + c] = x[u][ci];
                    }
                }
            } else if (d[u] == -1) {
#pragma unroll
                for (int ci = 0; ci < CH; ++ci) {
                    acc[ci][0] = fmaf(wj[u], bf16_lo(x[u][ci].x), acc[ci][0]); acc[ci][1] = fmaf(wj[u], bf16_hi(x[u][ci].x), acc[ci][1]);
                    acc[ci][2] = fmaf(wj[u], bf16_lo(x[u][ci].y), acc[ci][2]); acc[ci][3] = fmaf(wj[u], bf16_hi(x[u][ci].y), acc[ci][3]);
                    acc[ci][4] = fmaf(wj[u], bf16_lo(x[u][ci].z), acc[ci][4]); acc[ci][5] = fmaf(wj[u], bf16_hi(x[u][ci].z), acc[ci][5]);
                    acc[ci][6] = fmaf(wj[u], bf16_lo(x[u][ci].w), acc[ci][6]); acc[ci][7] = fmaf(wj[u], bf16_hi(x[u][ci].w), acc[ci][7]);
                }
            }
        }
    };
    {
        const int step = (int)gridDim.x * kG;
        int dA[kG], dB[kG];
        float wA[kG], wB[kG];
        uint4 xA[kG][CH], xB[kG][CH];
        int ib = cta * kG;
        load_group(ib, dA, wA, xA);
        for (; ib < i_hi; ib += 2 * step) {
            load_group(ib + step, dB, wB, xB);
            use_group(dA, wA, xA);
            load_group(ib + 2 * step, dA, wA, xA);
            use_group(dB, wB, xB);
        }
    }

    if (!w) return;                                           // no merged row in this mode
    // ---- clusters that touch the image span contribute a partial sum ---------------------------------
    const int cluster = cta / cl;
    const int q_first = 0, q_last = (int)gridDim.x / cl - 1;  // every cluster has seen merged rows
    const int rank = (int)hid_cluster_rank();
#pragma unroll
    for (int ci = 0; ci < CH; ++ci) {
        const int c = tid + ci * kHidThreads;
        if (c < V) {
            *reinterpret_cast<float4*>(s_sum + c * 8) = make_float4(acc[ci][0], acc[ci][1], acc[ci][2], acc[ci][3]);
            *reinterpret_cast<float4*>(s_sum + c * 8 + 4) = make_float4(acc[ci][4], acc[ci][5], acc[ci][6], acc[ci][7]);
        }
    }
    hid_cluster_barrier();
    if (rank == 0) {
        float* my_partial = partial + ((int64_t)b * gridDim.x / cl + cluster) * V * 8;
#pragma unroll
        for (int ci = 0; ci < CH; ++ci) {
            const int c = tid + ci * kHidThreads;
            if (c < V) {
                float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
                for (int r = 0; r < cl; ++r) {
                    const float4 a0 = hid_ld_cluster_f4(s_sum + c * 8, r), a1 = hid_ld_cluster_f4(s_sum + c * 8 + 4, r);
                    lo.x += a0.x; lo.y += a0.y; lo.z += a0.z; lo.w += a0.w;
                    hi.x += a1.x; hi.y += a1.y; hi.z += a1.z; hi.w += a1.w;
                }
                *reinterpret_cast<float4*>(my_partial + c * 8) = lo;
                *reinterpret_cast<float4*>(my_partial + c * 8 + 4) = hi;
            }
        }
    }
    // ---- the last cluster of this sequence finalises P_new, all of its CTAs sharing the columns -----------
    if (rank == 0) {
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int ticket = atomicAdd(&meta[b * kMetaInts + 1], 1);
            s_last = ticket == q_last - q_first;
        }
    }
    hid_cluster_barrier();                 // rank 0 has read every CTA's sums and knows whether we are last
    const int last = cl > 1 ? hid_ld_cluster_i32(&s_last, 0) : s_last;
    hid_cluster_barrier();                 // ... and everybody has asked it
    if (!last) return;
    __threadfence();
    const int nq = q_last - q_first + 1;                      // partials to add, in cluster order
    const int Vs = (V + cl - 1) / cl;                         // my slice of the column groups
    const int c_lo = min(V, rank * Vs), c_hi = min(V, c_lo + Vs);
    // two threads per column group, each adding half of the partials (four in flight); the halves are
    // added in order through shared memory
    const int hsel = tid >> 7, lane_c = tid & 127;
    const int q_mid = q_first + (nq + 1) / 2;
    const int qa = hsel ? q_mid : q_first, qb = hsel ? q_last + 1 : q_mid;
    float* s_fin = s_sum;                                     // [2][c_hi - c_lo][8], free after the barriers
    for (int cb = c_lo; cb < c_hi; cb += 128) {
        const int c = cb + lane_c;
        float t[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (c < c_hi) {
            for (int q = qa; q < qb; q += 4) {
                float4 lo[4], hi[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    lo[u] = hi[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (q + u < qb) {
                        const float4* pp = reinterpret_cast<const float4*>(
                            partial + ((int64_t)b * gridDim.x / cl + q + u) * V * 8 + c * 8);
                        lo[u] = __ldcg(pp); hi[u] = __ldcg(pp + 1);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    t[0] += lo[u].x; t[1] += lo[u].y; t[2] += lo[u].z; t[3] += lo[u].w;
                    t[4] += hi[u].x; t[5] += hi[u].y; t[6] += hi[u].z; t[7] += hi[u].w;
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) s_fin[(hsel * Vs + (c - c_lo)) * 8 + e] = t[e];
        }
    }
    __syncthreads();
    for (int c = c_lo + tid; c < c_hi; c += kHidThreads) {
        float t[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) t[e] = s_fin[(c - c_lo) * 8 + e] + s_fin[(Vs + (c - c_lo)) * 8 + e];
        uint4 o;
        o.x = pack_bf16(t[0], t[1]); o.y = pack_bf16(t[2], t[3]);
        o.z = pack_bf16(t[4], t[5]); o.w = pack_bf16(t[6], t[7]);
        hout[(int64_t)(i0 + k) * V + c] = o;
    }
    if (rank == 0 && tid == 0) meta[b * kMetaInts + 1] = 0;
}

template <int CH>
static lvlm_status launch_hidden_stream(const void* hidden, void* hidden_out, int64_t hid_sb, int64_t out_sb,
                                        const lvlm_dims* d, const HiddenGrid& L, const int32_t* dst_map,
                                        const float* wgt, int32_t* meta, float* partial, void* scratch,
                                        int64_t scr_sb, cudaStream_t stream) {
    const size_t smem = (size_t)L.V * 32 * (L.cl > 1 ? 1 : 2);      // the final sum needs two rows without a cluster
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(hidden_stream_kernel<CH>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    return launch_kernel(hidden_stream_kernel<CH>, dim3((unsigned)L.cps, (unsigned)d->B), dim3(kHidThreads), smem,
                         stream, L.cl, static_cast<const uint4*>(hidden), static_cast<uint4*>(hidden_out),
                         hid_sb / 8, out_sb / 8, L.V, d->N, d->i0, d->n, d->k, L.rpc, L.cl, dst_map, wgt, meta,
                         partial, static_cast<uint4*>(scratch), scr_sb / 8);
}

lvlm_status launch_hidden_rows(const void* hidden, void* hidden_out, int64_t hid_sb, int64_t out_sb,
                               const lvlm_dims* d, const HiddenGrid& L, const int32_t* dst_map,
                               const float* wgt, int32_t* meta, float* partial, void* scratch,
                               int64_t scr_sb, cudaStream_t stream) {
    const int chunks = (L.V + kHidThreads - 1) / kHidThreads;
    if (chunks > kHidMaxChunks) return LVLM_ERR_UNSUPPORTED;  // more than 8192 channels
    switch (chunks) {
        case 1: return launch_hidden_stream<1>(hidden, hidden_out, hid_sb, out_sb, d, L, dst_map, wgt, meta, partial, scratch, scr_sb, stream);
        case 2: return launch_hidden_stream<2>(hidden, hidden_out, hid_sb, out_sb, d, L, dst_map, wgt, meta, partial, scratch, scr_sb, stream);
        case 3: return launch_hidden_stream<3>(hidden, hidden_out, hid_sb, out_sb, d, L, dst_map, wgt, meta, partial, scratch, scr_sb, stream);
        case 4: return launch_hidden_stream<4>(hidden, hidden_out, hid_sb, out_sb, d, L, dst_map, wgt, meta, partial, scratch, scr_sb, stream);
    }
    return LVLM_ERR_UNSUPPORTED;
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_merge_compact(void* hidden, void* hidden_out, void* Kc, void* Vc,
                                           int32_t* pos_ids, const int32_t* rank,
                                           const lvlm_dims* d, lvlm_merge_mode mode,
                                           const float* w_custom, float* mass, int32_t* new_len,
                                           void* ws, size_t ws_bytes, int32_t* dev_status,
                                           void* stream_) {
    using namespace lvlm;
    (void)mass;
    cudaStream_t stream = (cudaStream_t)stream_;
    MergeLayout L;
    if (!hidden || !rank || !merge_layout(d, &L)) return LVLM_ERR_INVALID_ARG;
    if ((Kc == nullptr) != (Vc == nullptr)) return LVLM_ERR_INVALID_ARG;
    if ((int)mode < 0 || (int)mode > LVLM_W_NEAREST_KEPT) return LVLM_ERR_INVALID_ARG;
    if (mode == LVLM_W_CUSTOM && !w_custom) return LVLM_ERR_INVALID_ARG;
    if (Kc) {
        if (d->Hkv <= 0 || d->cap < d->N) return LVLM_ERR_INVALID_ARG;
        if (d->D != kHeadDim) return LVLM_ERR_UNSUPPORTED;
    }
    if (mode == LVLM_W_NEAREST_KEPT) {    // no P_new row: N - (n - k) rows come out
        L.r = d->n - d->k;
        L.Nout = d->N - L.r;
    }
    const int64_t hid_sb = d->hid_stride_b ? d->hid_stride_b : (int64_t)d->N * d->C;
    const int64_t out_sb = hidden_out ? (d->out_stride_b ? d->out_stride_b : (int64_t)L.Nout * d->C) : hid_sb;
    const int64_t kv_sh = d->kv_stride_h ? d->kv_stride_h : (int64_t)d->cap * d->D;
    const int64_t kv_sb = d->kv_stride_b ? d->kv_stride_b : (int64_t)d->Hkv * kv_sh;
    if (!aligned16(hidden) || !aligned16(hidden_out) || !aligned16(Kc) || !aligned16(Vc) ||
        hid_sb % 8 || out_sb % 8 || kv_sh % 8 || kv_sb % 8)
        return LVLM_ERR_ALIGNMENT;
    if (hid_sb < (int64_t)d->N * d->C || out_sb < (int64_t)L.Nout * d->C) return LVLM_ERR_INVALID_ARG;

    if (L.r <= 0) {                       // keep 100 %: every tensor stays as it is
        if (hidden_out && hidden_out != hidden) {
            LVLM_RETURN_IF_CUDA(cudaMemcpy2DAsync(hidden_out, out_sb * 2, hidden, hid_sb * 2,
                                                  (size_t)d->N * d->C * 2, d->B,
                                                  cudaMemcpyDeviceToDevice, stream));
        }
        if (new_len) return launch_kernel(identity_len_kernel, dim3((d->B + 127) / 128), dim3(128), 0, stream, 1,
                                          new_len, d->B, d->N);
        return LVLM_OK;
    }
    if (mode == LVLM_W_NEAREST_KEPT)
        return launch_nearest_kept(hidden, hidden_out, Kc, Vc, pos_ids, rank, d, mass, new_len, ws, ws_bytes,
                                   dev_status, stream);
    if (!ws || !aligned256(ws) || ws_bytes < L.total) return LVLM_ERR_WORKSPACE;
    char* wsb = static_cast<char*>(ws);
    int32_t* src_map = reinterpret_cast<int32_t*>(wsb + L.off_src);
    int32_t* dst_map = reinterpret_cast<int32_t*>(wsb + L.off_dst);
    float* wgt = reinterpret_cast<float*>(wsb + L.off_wgt);
    int32_t* meta = reinterpret_cast<int32_t*>(wsb + L.off_meta);
    float* partial = reinterpret_cast<float*>(wsb + L.off_partial);

    float inv_sum = 1.f;
    if (mode == LVLM_W_LINEAR_RANK) inv_sum = (float)(2.0 / ((double)L.r1 * ((double)L.r1 + 1.0)));
    else if (mode == LVLM_W_UNIFORM) inv_sum = (float)(1.0 / (double)L.r1);
    const int plan_threads = d->n >= 1024 ? 1024 : (d->n <= 128 ? 128 : ((d->n + 31) / 32) * 32);
    {
        int P = (d->n + 4095) / 4096;                    // CTAs per sequence: about four tiles of tokens each
        P = P < 1 ? 1 : (P > 8 ? 8 : P);
        const lvlm_status st = launch_kernel(merge_plan_kernel, dim3(P, d->B), dim3(plan_threads), 0, stream, P,
                                             rank, pos_ids, d->N, d->i0, d->n, d->k, (int)mode, inv_sum, w_custom,
                                             src_map, dst_map, wgt, meta, new_len, dev_status);
        if (st != LVLM_OK) return st;
    }

    if (hidden_out) {
        const lvlm_status st = launch_hidden_rows(hidden, hidden_out, hid_sb, out_sb, d, L.grid, dst_map, wgt, meta,
                                                  partial, nullptr, 0, stream);
        if (st != LVLM_OK) return st;
    } else {
        lvlm_status st = launch_inplace_compact(hidden, nullptr, hid_sb * 2, 0, d->B, 1, L.V,
                                                L.Nout, src_map, wgt, meta, d->N, d->n, d->i0,
                                                d->i0 + d->k, kMetaInts, stream, 1, -1, nullptr, dst_map);
        if (st != LVLM_OK) return st;
    }
    if (Kc) {
        lvlm_status st = launch_inplace_compact(Kc, Vc, kv_sb * 2, kv_sh * 2, d->B, d->Hkv,
                                                kHeadDim / 8, L.Nout, src_map, wgt, meta, d->N, d->n,
                                                d->i0, d->i0 + d->k, kMetaInts, stream, 1, -1, nullptr, dst_map);
        if (st != LVLM_OK) return st;
    }
    return LVLM_OK;
}
