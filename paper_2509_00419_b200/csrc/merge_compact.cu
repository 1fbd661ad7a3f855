// lvlm_merge_compact: P_new = W_v x P_merged and P_compressed = [P_unmerged, P_new]
// (Section 3.2.1, paragraph 4), applied to the hidden states, to that layer's K and V and
// to the position ids.
//
// Launches: (1) a plan kernel, one CTA per sequence, turns `rank` into a source-row map for
// every output row and a merge weight for every image token; (2) one streaming kernel moves
// the kept rows of the hidden states and accumulates the weighted sum of the merged rows
// (each input row is read once); (3) one kernel compacts K and V in place.
#include "common.cuh"
#include "compact.cuh"

namespace lvlm {

struct MergeLayout {
    int r1, r, Nout, V, colchunks, S;
    size_t off_src, off_wgt, off_meta, off_partial, total;
};

constexpr int kMergeThreads = 128;     // one 16-byte column group per thread in the merge part
constexpr int kMetaInts = 4;           // per sequence: first moved row, ticket counter, merged token, spare

static bool merge_layout(const lvlm_dims* d, MergeLayout* L) {
    if (!d || d->B <= 0 || d->N <= 0 || d->n <= 0 || d->C <= 0 || d->C % 8 || d->i0 < 0 ||
        d->k < 0 || d->k > d->n || (int64_t)d->i0 + d->n > d->N)
        return false;
    L->r1 = d->n - d->k;
    L->r = L->r1 > 0 ? L->r1 - 1 : 0;
    L->Nout = d->N - L->r;
    L->V = d->C / 8;
    L->colchunks = (L->V + kMergeThreads - 1) / kMergeThreads;
    int S = (4 * 148 + d->B * L->colchunks - 1) / (d->B * L->colchunks);
    const int max_by_rows = (d->n + 15) / 16;            // at least 16 image rows per slice
    S = S > max_by_rows ? max_by_rows : S;
    L->S = S < 1 ? 1 : (S > 128 ? 128 : S);
    size_t off = 0;
    L->off_src = off;     off = align_up(off + (size_t)d->B * d->N * 4, 256);
    L->off_wgt = off;     off = align_up(off + (size_t)d->B * d->n * 4, 256);
    L->off_meta = off;    off = align_up(off + (size_t)d->B * kMetaInts * 4, 256);
    L->off_partial = off; off = align_up(off + (size_t)d->B * L->S * d->C * 4, 256);
    L->total = off;
    return true;
}

size_t merge_compact_workspace(const lvlm_dims* d) {
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

// One CTA per sequence: source map, weights, position ids, new length.
__global__ void __launch_bounds__(1024)
merge_plan_kernel(const int32_t* __restrict__ rank, int32_t* pos_ids, int N, int i0, int n, int k,
                  int mode, float inv_sum, const float* __restrict__ w_custom,
                  int32_t* __restrict__ src_map, float* __restrict__ wgt,
                  int32_t* __restrict__ meta, int32_t* new_len, int32_t* dev_status) {
    __shared__ int scan_scratch[33];
    __shared__ float fsum_scratch[33];
    __shared__ int s_first_drop, s_merged_tok, s_pos_new;
    const int b = blockIdx.x;
    const int r1 = n - k, r = r1 - 1, Nout = N - r;
    const int32_t* rk = rank + (int64_t)b * n;
    int32_t* src = src_map + (int64_t)b * N;
    float* w = wgt + (int64_t)b * n;
    if (threadIdx.x == 0) { s_first_drop = n; s_merged_tok = 0; }

    if (mode == LVLM_W_CUSTOM) {
        float part = 0.f;
        for (int p = threadIdx.x; p < r1; p += blockDim.x) part += w_custom[p];
        const float tot = block_sum_fixed(part, fsum_scratch);
        inv_sum = 1.0f / tot;
    }
    __syncthreads();

    const int per = (n + blockDim.x - 1) / blockDim.x;
    const int j0 = min(n, (int)threadIdx.x * per), j1 = min(n, j0 + per);
    int cnt = 0, first_drop = n;
    bool bad = false;
    for (int j = j0; j < j1; ++j) {
        const int rj = rk[j];
        if (rj < 0 || rj >= n) bad = true;
        if (rj < k) ++cnt; else if (first_drop == n) first_drop = j;
        if (rj == k) s_merged_tok = j;
    }
    int total;
    int off = block_exclusive_scan(cnt, scan_scratch, &total);
    if (total != k) bad = true;
    if (first_drop < n) atomicMin(&s_first_drop, first_drop);
    for (int j = j0; j < j1; ++j) {
        const int rj = rk[j];
        float wj = 0.f;
        if (rj < k) {
            if (off < k) src[i0 + off] = i0 + j;
            ++off;
        } else {
            int p = rj - k;
            p = p < 0 ? 0 : (p >= r1 ? r1 - 1 : p);
            wj = merge_weight(mode, p, r1, inv_sum, w_custom);
        }
        w[j] = wj;
    }
    for (int o = threadIdx.x; o < Nout; o += blockDim.x) {
        if (o < i0) src[o] = o;
        else if (o == i0 + k) src[o] = -1;
        else if (o > i0 + k) src[o] = o + r;
    }
    if (bad && dev_status) atomicOr(dev_status, LVLM_DEV_BOUNDS);
    __syncthreads();
    if (threadIdx.x == 0) {
        meta[b * kMetaInts + 0] = i0 + s_first_drop;     // first row whose content changes
        meta[b * kMetaInts + 1] = 0;                     // ticket counter of the merge blocks
        meta[b * kMetaInts + 2] = s_merged_tok;
        if (new_len) new_len[b] = Nout;
        if (pos_ids) s_pos_new = pos_ids[(int64_t)b * N + i0 + s_merged_tok];
    }
    if (pos_ids) {
        // in place, tile by tile in increasing order: a tile's sources lie at or after it
        int32_t* pid = pos_ids + (int64_t)b * N;
        for (int o0 = 0; o0 < Nout; o0 += blockDim.x) {
            const int o = o0 + threadIdx.x;
            int val = 0;
            __syncthreads();
            if (o < Nout) { const int s = src[o]; val = s >= 0 ? pid[s] : s_pos_new; }
            __syncthreads();
            if (o < Nout) pid[o] = val;
        }
    }
}

__global__ void identity_len_kernel(int32_t* new_len, int B, int N) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) new_len[b] = N;
}

// Hidden states, out of place.  blockIdx.x < copy_blocks: move kept rows (one warp per output
// row, 16-byte vectors).  The remaining blocks each own a slice of the image rows and a chunk
// of 128 column groups, accumulate sum_j w_j x_j in fp32 in a fixed order and park the partial
// sum; the last block to finish for a sequence adds the partials in slice order, rounds once to
// bf16 and writes P_new.
__global__ void __launch_bounds__(256)
hidden_merge_compact_kernel(const uint4* __restrict__ hidden, uint4* __restrict__ out,
                            int64_t hid_stride_b, int64_t out_stride_b,   // in uint4
                            int V, int Nout, int i0, int n, int k,
                            const int32_t* __restrict__ src_map, int N,
                            const float* __restrict__ wgt, int32_t* meta,
                            float* partial, int S, int colchunks, int copy_blocks,
                            int rows_per_warp) {
    const int b = blockIdx.y;
    const uint4* hin = hidden + (int64_t)b * hid_stride_b;
    uint4* hout = out + (int64_t)b * out_stride_b;
    if ((int)blockIdx.x < copy_blocks) {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const int nwarp = blockDim.x >> 5;
        const int32_t* src = src_map + (int64_t)b * N;
        int o = ((int)blockIdx.x * nwarp + warp) * rows_per_warp;
        const int o_end = min(Nout, o + rows_per_warp);
        for (; o < o_end; ++o) {
            const int s = src[o];
            if (s < 0) continue;
            const uint4* srow = hin + (int64_t)s * V;
            uint4* drow = hout + (int64_t)o * V;
            int v = lane;
            for (; v + 96 < V; v += 128) {
                const uint4 a0 = __ldg(srow + v), a1 = __ldg(srow + v + 32);
                const uint4 a2 = __ldg(srow + v + 64), a3 = __ldg(srow + v + 96);
                drow[v] = a0; drow[v + 32] = a1; drow[v + 64] = a2; drow[v + 96] = a3;
            }
            for (; v < V; v += 32) drow[v] = __ldg(srow + v);
        }
        return;
    }
    // ---- merge part -------------------------------------------------------------------
    if (threadIdx.x >= kMergeThreads) return;
    const int mb = (int)blockIdx.x - copy_blocks;
    const int slice = mb / colchunks, chunk = mb % colchunks;
    const int cg = chunk * kMergeThreads + threadIdx.x;
    const int rows_per_slice = (n + S - 1) / S;
    const int j0 = min(n, slice * rows_per_slice), j1 = min(n, j0 + rows_per_slice);
    const float* w = wgt + (int64_t)b * n;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (cg < V) {
        const uint4* col = hin + (int64_t)i0 * V + cg;
        int j = j0;
        for (; j + 3 < j1; j += 4) {
            float wj[4];
            uint4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                wj[u] = w[j + u];
                x[u] = wj[u] != 0.f ? __ldg(col + (int64_t)(j + u) * V) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc[0] = fmaf(wj[u], bf16_lo(x[u].x), acc[0]); acc[1] = fmaf(wj[u], bf16_hi(x[u].x), acc[1]);
                acc[2] = fmaf(wj[u], bf16_lo(x[u].y), acc[2]); acc[3] = fmaf(wj[u], bf16_hi(x[u].y), acc[3]);
                acc[4] = fmaf(wj[u], bf16_lo(x[u].z), acc[4]); acc[5] = fmaf(wj[u], bf16_hi(x[u].z), acc[5]);
                acc[6] = fmaf(wj[u], bf16_lo(x[u].w), acc[6]); acc[7] = fmaf(wj[u], bf16_hi(x[u].w), acc[7]);
            }
        }
        for (; j < j1; ++j) {
            const float wj = w[j];
            if (wj == 0.f) continue;
            const uint4 x = __ldg(col + (int64_t)j * V);
            acc[0] = fmaf(wj, bf16_lo(x.x), acc[0]); acc[1] = fmaf(wj, bf16_hi(x.x), acc[1]);
            acc[2] = fmaf(wj, bf16_lo(x.y), acc[2]); acc[3] = fmaf(wj, bf16_hi(x.y), acc[3]);
            acc[4] = fmaf(wj, bf16_lo(x.z), acc[4]); acc[5] = fmaf(wj, bf16_hi(x.z), acc[5]);
            acc[6] = fmaf(wj, bf16_lo(x.w), acc[6]); acc[7] = fmaf(wj, bf16_hi(x.w), acc[7]);
        }
        float4* dst = reinterpret_cast<float4*>(partial + ((int64_t)(b * S + slice) * V + cg) * 8);
        dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    }
    // ---- last block of this sequence finalises P_new ------------------------------------
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int ticket = atomicAdd(&meta[b * kMetaInts + 1], 1);
        s_last = ticket == S * colchunks - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int c = threadIdx.x; c < V; c += kMergeThreads) {
        float t[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int s = 0; s < S; ++s) {
            const float4* p = reinterpret_cast<const float4*>(partial + ((int64_t)(b * S + s) * V + c) * 8);
            const float4 lo = __ldcg(p), hi = __ldcg(p + 1);
            t[0] += lo.x; t[1] += lo.y; t[2] += lo.z; t[3] += lo.w;
            t[4] += hi.x; t[5] += hi.y; t[6] += hi.z; t[7] += hi.w;
        }
        uint4 o;
        o.x = pack_bf16(t[0], t[1]); o.y = pack_bf16(t[2], t[3]);
        o.z = pack_bf16(t[4], t[5]); o.w = pack_bf16(t[6], t[7]);
        hout[(int64_t)(i0 + k) * V + c] = o;
    }
    if (threadIdx.x == 0) meta[b * kMetaInts + 1] = 0;
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
    if (mode == LVLM_W_NEAREST_KEPT) return LVLM_ERR_UNSUPPORTED;
    if (Kc) {
        if (d->Hkv <= 0 || d->cap < d->N) return LVLM_ERR_INVALID_ARG;
        if (d->D != kHeadDim) return LVLM_ERR_UNSUPPORTED;
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
        if (new_len) identity_len_kernel<<<(d->B + 127) / 128, 128, 0, stream>>>(new_len, d->B, d->N);
        return launch_status();
    }
    if (!ws || !aligned256(ws) || ws_bytes < L.total) return LVLM_ERR_WORKSPACE;
    char* wsb = static_cast<char*>(ws);
    int32_t* src_map = reinterpret_cast<int32_t*>(wsb + L.off_src);
    float* wgt = reinterpret_cast<float*>(wsb + L.off_wgt);
    int32_t* meta = reinterpret_cast<int32_t*>(wsb + L.off_meta);
    float* partial = reinterpret_cast<float*>(wsb + L.off_partial);

    float inv_sum = 1.f;
    if (mode == LVLM_W_LINEAR_RANK) inv_sum = (float)(2.0 / ((double)L.r1 * ((double)L.r1 + 1.0)));
    else if (mode == LVLM_W_UNIFORM) inv_sum = (float)(1.0 / (double)L.r1);
    const int plan_threads = d->n >= 1024 ? 1024 : (d->n <= 128 ? 128 : ((d->n + 31) / 32) * 32);
    merge_plan_kernel<<<d->B, plan_threads, 0, stream>>>(rank, pos_ids, d->N, d->i0, d->n, d->k,
                                                         (int)mode, inv_sum, w_custom, src_map, wgt,
                                                         meta, new_len, dev_status);
    if (cudaGetLastError() != cudaSuccess) return LVLM_ERR_CUDA;

    if (hidden_out) {
        // rows per warp chosen so that the grid has a few CTAs per SM when the job allows
        const int warps = 8;
        int rpw = (int)(((int64_t)d->B * L.Nout + 8 * 148 * warps - 1) / (8 * 148 * warps));
        rpw = rpw < 1 ? 1 : (rpw > 4 ? 4 : rpw);
        const int copy_blocks = (L.Nout + warps * rpw - 1) / (warps * rpw);
        dim3 grid(copy_blocks + L.S * L.colchunks, d->B);
        hidden_merge_compact_kernel<<<grid, 256, 0, stream>>>(
            static_cast<const uint4*>(hidden), static_cast<uint4*>(hidden_out), hid_sb / 8, out_sb / 8,
            L.V, L.Nout, d->i0, d->n, d->k, src_map, d->N, wgt, meta, partial, L.S, L.colchunks,
            copy_blocks, rpw);
        if (cudaGetLastError() != cudaSuccess) return LVLM_ERR_CUDA;
    } else {
        lvlm_status st = launch_inplace_compact(hidden, nullptr, hid_sb * 2, 0, d->B, 1, L.V,
                                                L.Nout, src_map, wgt, meta, d->N, d->n, d->i0,
                                                d->i0 + d->k, kMetaInts, stream);
        if (st != LVLM_OK) return st;
    }
    if (Kc) {
        lvlm_status st = launch_inplace_compact(Kc, Vc, kv_sb * 2, kv_sh * 2, d->B, d->Hkv,
                                                kHeadDim / 8, L.Nout, src_map, wgt, meta, d->N, d->n,
                                                d->i0, d->i0 + d->k, kMetaInts, stream);
        if (st != LVLM_OK) return st;
    }
    return LVLM_OK;
}
