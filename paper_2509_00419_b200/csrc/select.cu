// lvlm_select_topk: total order of the image tokens by (score descending, index ascending).
// Section 3.2.1, paragraph 4: the tokens with the highest scores form P_unmerged, the others
// form P_merged, "reordered by their importance".
//
// The rank of a token is the number of tokens that come before it in that order, so it can be
// counted directly: nothing iterative, every token independent of the others.  Keys are 64-bit
// (order-preserving image of the score << 32 | index), so the order is total and ties go to the
// lower index.  grid (blocks of 256 tokens, S, B): a CTA counts, for its 256 tokens, the keys of
// one slice of the sequence that are smaller (shared memory, every thread reads the same key at
// the same time); the S CTAs of a cluster add their counts through distributed shared memory.
// The optional outputs (kept list, near-tie count) come from a second, small kernel.
#include "common.cuh"
#include "rank_count.cuh"

namespace lvlm {

// grid (blocks of 256 jt tokens, S, B), clusters (1, S, 1).
__global__ void __launch_bounds__(kRankThreads)
select_count_kernel(const float* __restrict__ score, int64_t stride, int n, int S, int slice_len, int jt,
                    int32_t* __restrict__ rank, int32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_cnt[kRankMaxJT * kRankThreads];
    pdl_enter();
    const int b = blockIdx.z;
    const float* row = score + (int64_t)b * stride;
    bool nonfinite = false;
    auto key_of = [&](int i) { return ((uint64_t)desc_key(row[i], &nonfinite) << 32) | (uint32_t)i; };
    int cnt[kRankMaxJT];
    if (rank_by_counting(key_of, n, S, slice_len, jt, reinterpret_cast<uint64_t*>(smem_raw), s_cnt, cnt)) {
#pragma unroll
        for (int u = 0; u < kRankMaxJT; ++u) {
            const int j = rank_key_index(jt, u);
            if (u < jt && j < n) rank[(int64_t)b * n + j] = cnt[u];
        }
    }
    // every key is looked at by the CTAs of slice 0 as "their own" key: one report is enough
    if (nonfinite && blockIdx.y == 0 && dev_status) atomicOr(dev_status, LVLM_DEV_NONFINITE);
}

// One CTA per sequence: the kept tokens in ascending order (prefix sum of rank < k over the index) and
// the number of near-ties among neighbours (p, p+1) of the order with p+1 >= k.
__global__ void __launch_bounds__(1024)
select_aux_kernel(const float* __restrict__ score, int64_t stride, int n, int k,
                  const int32_t* __restrict__ rank, int32_t* __restrict__ kept_idx,
                  int32_t* __restrict__ near_tie) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int32_t* order = reinterpret_cast<int32_t*>(smem_raw);           // [n] token at every place of the order
    __shared__ int scan_scratch[33];
    __shared__ int s_near;
    pdl_enter();
    const int b = blockIdx.x;
    const float* row = score + (int64_t)b * stride;
    const int32_t* rk = rank + (int64_t)b * n;
    if (threadIdx.x == 0) s_near = 0;
    for (int j = threadIdx.x; j < n; j += blockDim.x) {
        const int p = rk[j];
        if (p >= 0 && p < n) order[p] = j;
    }
    __syncthreads();
    if (near_tie) {
        int near = 0;
        for (int p = threadIdx.x + max(k - 1, 0); p + 1 < n; p += blockDim.x) {
            const float a = row[order[p]], c = row[order[p + 1]];
            const float dgap = __fsub_rn(a, c);
            const float t = __fmul_rn(1e-4f, fabsf(a));
            if (dgap < t) ++near;
        }
        near = warp_sum(near);
        if ((threadIdx.x & 31) == 0 && near) atomicAdd(&s_near, near);
        __syncthreads();
        if (threadIdx.x == 0) near_tie[b] = s_near;
    }
    if (kept_idx && k > 0) {
        const int per = (n + blockDim.x - 1) / blockDim.x;
        const int j0 = min(n, (int)threadIdx.x * per), j1 = min(n, j0 + per);
        int cnt = 0;
        for (int j = j0; j < j1; ++j) cnt += rk[j] < k;
        int total;
        int off = block_exclusive_scan(cnt, scan_scratch, &total);
        for (int j = j0; j < j1; ++j)
            if (rk[j] < k && off < k) kept_idx[(int64_t)b * k + off++] = j;
    }
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_select_topk(const float* score, int B, int n, int64_t score_stride,
                                         int k, int32_t* rank, int32_t* kept_idx,
                                         int32_t* near_tie, void* ws, size_t ws_bytes,
                                         int32_t* dev_status, void* stream_) {
    using namespace lvlm;
    (void)ws; (void)ws_bytes;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!score || !rank || B <= 0 || n <= 0 || k < 0 || k > n) return LVLM_ERR_INVALID_ARG;
    if (score_stride == 0) score_stride = n;
    if (score_stride < n) return LVLM_ERR_INVALID_ARG;
    if (n > kRankMaxKeys) return LVLM_ERR_UNSUPPORTED;
    if ((kept_idx || near_tie) && (size_t)n * 4 > (size_t)kMaxDynSmem) return LVLM_ERR_UNSUPPORTED;
    int S, slice_len, jt;
    rank_shape(n, B, &S, &slice_len, &jt);
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(select_count_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    {
        const lvlm_status st = launch_kernel_cluster(select_count_kernel, dim3((n + kRankThreads * jt - 1) / (kRankThreads * jt), S, B),
                                                     dim3(kRankThreads), rank_smem_bytes(slice_len), stream, dim3(1, S, 1),
                                                     score, score_stride, n, S, slice_len, jt, rank, dev_status);
        if (st != LVLM_OK) return st;
    }
    if (!kept_idx && !near_tie) return LVLM_OK;
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(select_aux_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    const int threads = n >= 1024 ? 1024 : ((n + 31) / 32) * 32;
    return launch_kernel(select_aux_kernel, dim3(B), dim3(threads), (size_t)n * 4, stream, 1,
                         score, score_stride, n, k, rank, kept_idx, near_tie);
}
