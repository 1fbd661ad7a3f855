// lvlm_select_topk: total order of the image tokens by (score descending, index ascending).
// Section 3.2.1, paragraph 4: the tokens with the highest scores form P_unmerged, the others
// form P_merged, "reordered by their importance".
#include "common.cuh"
#include "sort.cuh"

namespace lvlm {

// One CTA per sequence.  Shared memory: P 64-bit keys (score key << 32 | index) followed by
// n int32 ranks.  The stable order falls out of the index in the low word.
__global__ void __launch_bounds__(1024)
select_rank_kernel(const float* __restrict__ score, int64_t stride, int n, int k, int P,
                   int32_t* __restrict__ rank, int32_t* __restrict__ kept_idx,
                   int32_t* __restrict__ near_tie, int32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* keys = reinterpret_cast<uint64_t*>(smem_raw);
    int32_t* srank = reinterpret_cast<int32_t*>(keys + P);
    __shared__ int scan_scratch[33];
    __shared__ int s_near;

    pdl_enter();
    const int b = blockIdx.x;
    const float* row = score + (int64_t)b * stride;
    bool nonfinite = false;
    if (threadIdx.x == 0) s_near = 0;
    for (int j = threadIdx.x; j < P; j += blockDim.x) {
        uint64_t key = ~0ull;
        if (j < n) key = ((uint64_t)desc_key(row[j], &nonfinite) << 32) | (uint32_t)j;
        keys[j] = key;
    }
    if (nonfinite && dev_status) atomicOr(dev_status, LVLM_DEV_NONFINITE);
    __syncthreads();
    block_bitonic_sort(keys, P);

    int near = 0;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        const int idx = (int)(uint32_t)keys[p];
        srank[idx] = p;
        rank[(int64_t)b * n + idx] = p;
        if (near_tie && p + 1 >= k && p + 1 < n) {
            const float a = row[idx];
            const float c = row[(int)(uint32_t)keys[p + 1]];
            const float dgap = __fsub_rn(a, c);
            const float t = __fmul_rn(1e-4f, fabsf(a));
            if (dgap < t) ++near;
        }
    }
    if (near_tie) {
        near = warp_sum(near);
        if ((threadIdx.x & 31) == 0 && near) atomicAdd(&s_near, near);
    }
    __syncthreads();
    if (near_tie && threadIdx.x == 0) near_tie[b] = s_near;

    if (kept_idx && k > 0) {
        // kept tokens in ascending index order: prefix sum of (rank < k) over the index
        const int per = (n + blockDim.x - 1) / blockDim.x;
        const int j0 = min(n, (int)threadIdx.x * per), j1 = min(n, j0 + per);
        int cnt = 0;
        for (int j = j0; j < j1; ++j) cnt += srank[j] < k;
        int total;
        int off = block_exclusive_scan(cnt, scan_scratch, &total);
        for (int j = j0; j < j1; ++j)
            if (srank[j] < k) kept_idx[(int64_t)b * k + off++] = j;
    }
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_select_topk(const float* score, int B, int n, int64_t score_stride,
                                         int k, int32_t* rank, int32_t* kept_idx,
                                         int32_t* near_tie, void* ws, size_t ws_bytes,
                                         int32_t* dev_status, void* stream) {
    using namespace lvlm;
    (void)ws; (void)ws_bytes;
    if (!score || !rank || B <= 0 || n <= 0 || k < 0 || k > n) return LVLM_ERR_INVALID_ARG;
    if (score_stride == 0) score_stride = n;
    if (score_stride < n) return LVLM_ERR_INVALID_ARG;
    if (n > kMaxSortN) return LVLM_ERR_UNSUPPORTED;
    const int P = next_pow2(n < 2 ? 2 : n);
    int threads = P / 2;
    threads = threads < 32 ? 32 : (threads > 1024 ? 1024 : threads);
    const size_t smem = (size_t)P * 8 + (size_t)n * 4;
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(select_rank_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    return launch_kernel(select_rank_kernel, dim3(B), dim3(threads), smem, (cudaStream_t)stream, 1,
                         score, score_stride, n, k, P, rank, kept_idx, near_tie, dev_status);
}
