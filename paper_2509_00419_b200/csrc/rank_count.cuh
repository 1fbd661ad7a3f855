// Rank by counting: the place of a key in the ascending order of distinct 64-bit keys is the
// number of keys smaller than it.  Shared by token selection and by the grouping step of the
// nearest-kept merge.  A CTA holds one slice of the keys in shared memory and every thread counts
// for its own key; the CTAs of a cluster (one per slice, along y) add their counts through
// distributed shared memory.
#pragma once
#include "common.cuh"

namespace lvlm {

constexpr int kRankThreads = 256;
constexpr int kRankMaxCluster = 8;
constexpr int kRankMaxSlice = 16384;       // keys of one slice in shared memory (128 KB)
constexpr int kRankMaxKeys = kRankMaxCluster * kRankMaxSlice;     // 131072 keys per sequence

__device__ __forceinline__ uint32_t rank_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void rank_cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ int rank_ld_cluster(const int* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    int v;
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}

// Number of slices (cluster size) and keys per slice for n keys in each of B sequences: up to eight
// CTAs of 256 threads per SM, at least 256 keys per slice; the slice length is even.
inline void rank_shape(int n, int B, int* S, int* slice_len) {
    const int jblocks = (n + kRankThreads - 1) / kRankThreads;
    int s = 1;
    while (s < kRankMaxCluster && (int64_t)jblocks * B * (2 * s) <= 8 * 148 && n / (2 * s) >= 256) s *= 2;
    while (s < kRankMaxCluster && (n + s - 1) / s > kRankMaxSlice) s *= 2;       // a slice has to fit
    *S = s;
    *slice_len = (((n + s - 1) / s) + 1) & ~1;
}

// Call from every thread of a CTA of kRankThreads threads in a grid (key blocks, S, B) with clusters
// (1, S, 1).  key_of(i) gives key i of this sequence (i < n).  Returns true in the threads that hold a
// final count (*count = number of keys smaller than key j, j = blockIdx.x * 256 + threadIdx.x < n).
template <typename KeyFn>
__device__ __forceinline__ bool rank_by_counting(KeyFn key_of, int n, int S, int slice_len, uint64_t* sk,
                                                 int* s_cnt, int* count) {
    const int s = (int)rank_cluster_rank(), tid = threadIdx.x;
    const int i_lo = s * slice_len;
    for (int i = tid; i < slice_len; i += kRankThreads) {
        const int gi = i_lo + i;
        sk[i] = gi < n ? key_of(gi) : ~0ull;              // padding sorts after every real key
    }
    const int j = blockIdx.x * kRankThreads + tid;
    const uint64_t kj = j < n ? key_of(j) : 0ull;
    __syncthreads();
    int cnt = 0;
    const ulonglong2* sk2 = reinterpret_cast<const ulonglong2*>(sk);
#pragma unroll 4
    for (int i = 0; i < slice_len / 2; ++i) {
        const ulonglong2 v = sk2[i];
        cnt += (v.x < kj) + (v.y < kj);
    }
    if (S == 1) { *count = cnt; return j < n; }
    s_cnt[tid] = cnt;
    rank_cluster_barrier();
    bool mine = false;
    if (s == 0 && j < n) {
        int tot = 0;
        for (int r = 0; r < S; ++r) tot += rank_ld_cluster(&s_cnt[tid], r);
        *count = tot;
        mine = true;
    }
    rank_cluster_barrier();                               // nobody leaves while its counts are read
    return mine;
}

}  // namespace lvlm
