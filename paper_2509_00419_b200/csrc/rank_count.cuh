// Rank by counting: the place of a key in the ascending order of distinct 64-bit keys is the
// number of keys smaller than it.  Shared by token selection and by the grouping step of the
// nearest-kept merge.  A CTA holds one slice of the keys in shared memory and every thread counts
// for its own key; the CTAs of a cluster (one per slice, along y) add their counts through
// distributed shared memory.  A short slice is simply read through.  A long slice is first put into
// 1024 bins - linear in the high word of the key, or, where that leaves a bin deeper than 256 keys (ties, a
// handful of distinct scores), bounded by a sorted sample of the slice's own keys: the keys are distinct
// (the index is their low word), so such bins stay a few keys deep whatever the scores look like.  All
// keys of lower bins are smaller, so only the thread's own bin is read through; how the keys happen to
// be ordered inside a bin does not matter, the count is the same.
#pragma once
#include "common.cuh"

namespace lvlm {

constexpr int kRankThreads = 256;
constexpr int kRankMaxCluster = 8;
constexpr int kRankMaxSlice = 8192;        // keys of one slice in shared memory (twice 64 KB when binned)
constexpr int kRankMaxKeys = kRankMaxCluster * kRankMaxSlice;     // 65536 keys per sequence
constexpr int kRankBinFrom = 1024;         // slices at least this long are binned
constexpr int kRankBins = 1024;
constexpr int kRankMaxJT = 4;              // keys a thread ranks when the slices are binned (bins are built once per CTA)

// Shared memory a CTA needs for a slice of slice_len keys.
inline size_t rank_smem_bytes(int slice_len) {
    return slice_len >= kRankBinFrom ? (size_t)slice_len * 16 + (size_t)kRankBins * 8 + (size_t)(2 * kRankBins + 2) * 4
                                     : (size_t)slice_len * 8;
}

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

// Ascending sort of P (a power of two) 64-bit keys in shared memory by the whole CTA.
__device__ __forceinline__ void rank_bitonic_sort(uint64_t* keys, int P) {
    for (int k2 = 2; k2 <= P; k2 <<= 1) {
        for (int j = k2 >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < (P >> 1); t += blockDim.x) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const int l = i | j;
                const bool up = (i & k2) == 0;
                const uint64_t a = keys[i], b = keys[l];
                if ((a > b) == up) { keys[i] = b; keys[l] = a; }
            }
            __syncthreads();
        }
    }
}

// Number of slices (cluster size) and keys per slice for n keys in each of B sequences: up to eight
// CTAs of 256 threads per SM, at least 256 keys per slice; the slice length is even.
inline void rank_shape(int n, int B, int* S, int* slice_len, int* jt) {
    const int jblocks = (n + kRankThreads - 1) / kRankThreads;
    int s = 1;
    while (s < kRankMaxCluster && (int64_t)jblocks * B * (2 * s) <= 8 * 148 && n / (2 * s) >= 256) s *= 2;
    while (s < kRankMaxCluster && (n + s - 1) / s > kRankMaxSlice) s *= 2;       // a slice has to fit
    *S = s;
    *slice_len = (((n + s - 1) / s) + 1) & ~1;
    *jt = *slice_len >= 4096 ? kRankMaxJT : 1;           // few CTAs per slice when a slice is costly to bin
}

// Call from every thread of a CTA of kRankThreads threads in a grid (ceil(n / (256 jt)), S, B) with
// clusters (1, S, 1).  key_of(i) gives key i of this sequence (i < n).  A thread ranks the jt keys
// j_u = rank_key_index(u) = (blockIdx.x * jt + u) * 256 + threadIdx.x.  Returns true in the threads that
// hold final counts (count[u] = number of keys smaller than key j_u, for the j_u < n).
// s_cnt: kRankMaxJT * kRankThreads ints of shared memory.
__device__ __forceinline__ int rank_key_index(int jt, int u) { return (blockIdx.x * jt + u) * kRankThreads + threadIdx.x; }

template <typename KeyFn>
__device__ __forceinline__ bool rank_by_counting(KeyFn key_of, int n, int S, int slice_len, int jt, uint64_t* sk,
                                                 int* s_cnt, int* count) {
    const int s = (int)rank_cluster_rank(), tid = threadIdx.x;
    const int i_lo = s * slice_len;
    for (int i = tid; i < slice_len; i += kRankThreads) {
        const int gi = i_lo + i;
        sk[i] = gi < n ? key_of(gi) : ~0ull;              // padding sorts after every real key
    }
    uint64_t kjs[kRankMaxJT];
#pragma unroll
    for (int u = 0; u < kRankMaxJT; ++u) {
        const int j = rank_key_index(jt, u);
        kjs[u] = (u < jt && j < n) ? key_of(j) : 0ull;
        count[u] = 0;
    }
    __syncthreads();
    if (slice_len >= kRankBinFrom) {
        __shared__ int s_scan[33];
        __shared__ uint32_t s_min[kRankThreads / 32], s_max[kRankThreads / 32];
        __shared__ int s_deepest;
        uint64_t* sb = sk + slice_len;                                   // the keys again, bin by bin
        uint64_t* spl = sb + slice_len;                                  // [kRankBins] sorted sample: bin boundaries
        int* start = reinterpret_cast<int*>(spl + kRankBins);            // [kRankBins + 1]
        int* cursor = start + kRankBins + 1;                             // [kRankBins]
        const int nvalid = max(0, min(slice_len, n - i_lo));
        // First try: bins linear in the high word between the slice's extremes (one multiply per key).
        uint32_t lo = 0xFFFFFFFFu, hi = 0u;
        for (int i = tid; i < nvalid; i += kRankThreads) {
            const uint32_t h = (uint32_t)(sk[i] >> 32);
            lo = min(lo, h); hi = max(hi, h);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = min(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
            hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
        }
        if ((tid & 31) == 0) { s_min[tid >> 5] = lo; s_max[tid >> 5] = hi; }
        if (tid == 0) s_deepest = 0;
        for (int i = tid; i <= kRankBins; i += kRankThreads) start[i] = 0;
        __syncthreads();
#pragma unroll
        for (int wv = 0; wv < kRankThreads / 32; ++wv) { lo = min(lo, s_min[wv]); hi = max(hi, s_max[wv]); }
        const uint64_t span = (uint64_t)(hi - lo) + 1;                   // hi >= lo whenever the slice has keys
        auto bin_linear = [&](uint64_t key) {
            const uint32_t h = (uint32_t)(key >> 32);
            if (h <= lo) return 0;
            if (h >= hi) return kRankBins - 1;
            return (int)(((uint64_t)(h - lo) * kRankBins) / span);
        };
        // bin of a key = number of boundaries spl[1..1023] that are <= key (binary search), 0 .. 1023
        auto bin_sampled = [&](uint64_t key) {
            int lo_i = 0, hi_i = kRankBins - 1;                          // boundaries spl[1 + lo_i .. 1 + hi_i)
            while (lo_i < hi_i) {
                const int mid = (lo_i + hi_i) >> 1;
                if (spl[1 + mid] <= key) lo_i = mid + 1; else hi_i = mid;
            }
            return lo_i;
        };
        for (int i = tid; i < nvalid; i += kRankThreads) {
            const int c = atomicAdd(&start[bin_linear(sk[i])], 1) + 1;
            if (c > 256) atomicMax(&s_deepest, c);                       // (rarely taken)
        }
        __syncthreads();
        // Scores that pile up in a few values (ties, a handful of distinct numbers) would make a bin as deep as the
        // slice.  Then the bins are rebuilt with boundaries taken from a sorted sample of the slice's own keys:
        // the keys are distinct (the index is their low word), so those bins are a few keys deep whatever
        // the scores look like.
        const bool sampled = s_deepest > 256;
        __syncthreads();
        if (sampled) {
            for (int t = tid; t < kRankBins; t += kRankThreads) {
                const int i = nvalid >= kRankBins ? (int)(((int64_t)t * nvalid) / kRankBins) : t;
                spl[t] = i < nvalid ? sk[i] : ~0ull;                     // padding sorts last and bounds nothing
            }
            for (int i = tid; i <= kRankBins; i += kRankThreads) start[i] = 0;
            __syncthreads();
            rank_bitonic_sort(spl, kRankBins);
            for (int i = tid; i < nvalid; i += kRankThreads) atomicAdd(&start[bin_sampled(sk[i])], 1);
            __syncthreads();
        }
        auto bin_of = [&](uint64_t key) { return sampled ? bin_sampled(key) : bin_linear(key); };
        {   // exclusive scan of the bin counts: four bins per thread
            int c4[4], sum = 0;
#pragma unroll
            for (int u = 0; u < 4; ++u) { c4[u] = start[tid * 4 + u]; sum += c4[u]; }
            int total;
            int run = block_exclusive_scan(sum, s_scan, &total);
#pragma unroll
            for (int u = 0; u < 4; ++u) { start[tid * 4 + u] = run; cursor[tid * 4 + u] = run; run += c4[u]; }
            if (tid == 0) start[kRankBins] = total;
        }
        __syncthreads();
        for (int i = tid; i < nvalid; i += kRankThreads) {
            const uint64_t key = sk[i];
            sb[atomicAdd(&cursor[bin_of(key)], 1)] = key;
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < kRankMaxJT; ++u) {
            const uint64_t kj = kjs[u];
            int cnt = 0;
            if (nvalid > 0 && u < jt && rank_key_index(jt, u) < n) {
                const int bj = bin_of(kj);
                cnt = start[bj];
                for (int p = start[bj]; p < start[bj + 1]; ++p) cnt += sb[p] < kj;
            }
            count[u] = cnt;
        }
    } else {
        const uint64_t kj = kjs[0];                       // short slices: one key per thread (jt == 1)
        int cnt = 0;
        const ulonglong2* sk2 = reinterpret_cast<const ulonglong2*>(sk);
#pragma unroll 4
        for (int i = 0; i < slice_len / 2; ++i) {
            const ulonglong2 v = sk2[i];
            cnt += (v.x < kj) + (v.y < kj);
        }
        count[0] = cnt;
    }
    if (S == 1) return true;
#pragma unroll
    for (int u = 0; u < kRankMaxJT; ++u) s_cnt[u * kRankThreads + tid] = count[u];
    rank_cluster_barrier();
    const bool mine = s == 0;
    if (mine) {
#pragma unroll
        for (int u = 0; u < kRankMaxJT; ++u) {
            int tot = 0;
            if (u < jt)
                for (int r = 0; r < S; ++r) tot += rank_ld_cluster(&s_cnt[u * kRankThreads + tid], r);
            count[u] = tot;
        }
    }
    rank_cluster_barrier();                               // nobody leaves while its counts are read
    return mine;
}

}  // namespace lvlm
