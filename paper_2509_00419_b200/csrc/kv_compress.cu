// lvlm_kv_compress: per (sequence, KV head) eviction of low-score cache entries
// (Section 3.2.2, paragraph 2: sort the scores in descending order, keep the entries whose
// accumulated score reaches the threshold beta, discard the other image entries; Appendix A.2:
// beta = 0.995).  A plan kernel ranks the evictable entries, finds the count, builds the
// survivor map and compacts the small per-entry arrays; the shared in-place compaction kernel
// then moves the K and V rows.
#include "common.cuh"
#include "compact.cuh"
#include "sort.cuh"

namespace lvlm {

struct KvLayout { size_t off_src, off_meta, off_nout, total; };

static bool kv_layout(const lvlm_dims* d, KvLayout* L) {
    if (!d || d->B <= 0 || d->Hkv <= 0 || d->cap <= 0 || d->recent < 0) return false;
    size_t off = 0;
    const size_t heads = (size_t)d->B * d->Hkv;
    L->off_src = off;  off = align_up(off + heads * d->cap * 4, 256);
    L->off_meta = off; off = align_up(off + heads * 4, 256);
    L->off_nout = off; off = align_up(off + heads * 4, 256);
    L->total = off;
    return true;
}

size_t kv_compress_workspace(const lvlm_dims* d) {
    KvLayout L;
    return kv_layout(d, &L) ? L.total : 0;
}

// Exclusive prefix sum of one 64-bit integer per thread (same contract as block_exclusive_scan).
__device__ __forceinline__ long long block_exclusive_scan_ll(long long v, long long* scratch,
                                                             long long* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    long long incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        long long w = lane < nwarp ? scratch[lane] : 0;
        long long wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            long long t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += t;
        }
        scratch[lane] = wi - w;
        if (lane == 31) scratch[32] = wi;
    }
    __syncthreads();
    *total = scratch[32];
    return scratch[warp] + incl - v;
}

// Score in integer units of 2^-24 (negative and non-finite scores count as zero).
__device__ __forceinline__ long long score_units(float s) {
    if (!(s > 0.f) || (__float_as_uint(s) & 0x7F800000u) == 0x7F800000u) return 0;
    return __float2ll_rn(ldexpf(s, 24));
}

// ceil(a * b / c) for a, b < 2^63, c = 10^6, in 128-bit arithmetic.
__device__ __forceinline__ unsigned long long ceil_muldiv(unsigned long long a, unsigned long long b,
                                                          unsigned long long c) {
    unsigned long long hi = __umul64hi(a, b), lo = a * b;
    // long division of (hi:lo) by c, 64 steps; hi < c holds because a < c (beta < 1) ... not
    // assumed: reduce hi first.
    unsigned long long rem = hi % c;
    unsigned long long q = 0;
    for (int bit = 63; bit >= 0; --bit) {
        rem = (rem << 1) | ((lo >> bit) & 1ull);        // rem < 2c < 2^63, no overflow
        q <<= 1;
        if (rem >= c) { rem -= c; q |= 1ull; }
    }
    // the quotient's high word (hi / c) is zero whenever a <= c, which the caller guarantees
    return q + (rem != 0);
}

constexpr int kPlanBins = 1024;
constexpr int kPlanBinFrom = 512;          // evictable sets at least this large are ordered by binned counting
constexpr int kPlanBinMaxCap = 8192;       // ... when the second key array fits in shared memory

// Ascending order of m distinct 64-bit keys (m <= blockDim.x * 16) without a sorting network: the keys
// are put into 1024 bins by their high word (linear between the extremes), the place of a key is the
// number of keys in lower bins plus the number of smaller keys in its own bin.  On return `sorted` holds
// the keys in order.  srank: m ints, bins: 2 * kPlanBins + 1 ints of shared memory.
__device__ __forceinline__ void block_order_by_bins(const uint64_t* keys, uint64_t* sorted, int m, int* srank,
                                                    int* bins, int* scan_scratch) {
    __shared__ uint32_t s_min[32], s_max[32];
    int* start = bins;                       // [kPlanBins + 1]
    int* cursor = bins + kPlanBins + 1;      // [kPlanBins]
    const int tid = threadIdx.x;
    uint32_t lo = 0xFFFFFFFFu, hi = 0u;
    for (int i = tid; i < m; i += blockDim.x) {
        const uint32_t h = (uint32_t)(keys[i] >> 32);
        lo = min(lo, h); hi = max(hi, h);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = min(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
        hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
    }
    if ((tid & 31) == 0) { s_min[tid >> 5] = lo; s_max[tid >> 5] = hi; }
    for (int i = tid; i <= kPlanBins; i += blockDim.x) start[i] = 0;
    __syncthreads();
    for (int wv = 0; wv < (int)(blockDim.x >> 5); ++wv) { lo = min(lo, s_min[wv]); hi = max(hi, s_max[wv]); }
    const uint64_t span = (uint64_t)(hi - lo) + 1;
    auto bin_of = [&](uint32_t h) { return (int)(((uint64_t)(h - lo) * kPlanBins) / span); };
    for (int i = tid; i < m; i += blockDim.x) atomicAdd(&start[bin_of((uint32_t)(keys[i] >> 32))], 1);
    __syncthreads();
    {   // exclusive scan of the bin counts: the first 256 threads take four bins each
        int c4[4] = {0, 0, 0, 0}, sum = 0;
        if (tid < kPlanBins / 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) { c4[u] = start[tid * 4 + u]; sum += c4[u]; }
        }
        int total;
        int run = block_exclusive_scan(sum, scan_scratch, &total);
        if (tid < kPlanBins / 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) { start[tid * 4 + u] = run; cursor[tid * 4 + u] = run; run += c4[u]; }
        }
        if (tid == 0) start[kPlanBins] = total;
    }
    __syncthreads();
    for (int i = tid; i < m; i += blockDim.x) {
        const uint64_t key = keys[i];
        sorted[atomicAdd(&cursor[bin_of((uint32_t)(key >> 32))], 1)] = key;       // bin by bin, any order inside
    }
    __syncthreads();
    for (int i = tid; i < m; i += blockDim.x) {
        const uint64_t key = keys[i];
        const int bj = bin_of((uint32_t)(key >> 32));
        int r = start[bj];
        for (int p = start[bj]; p < start[bj + 1]; ++p) r += sorted[p] < key;
        srank[i] = r;
    }
    __syncthreads();
    for (int i = tid; i < m; i += blockDim.x) sorted[srank[i]] = keys[i];
    __syncthreads();
}

__global__ void __launch_bounds__(1024)
kv_plan_kernel(float* acc_score, int32_t* pos, int32_t* len, const int32_t* __restrict__ e_lo,
               const int32_t* __restrict__ e_hi, int Hkv, int cap, int recent, int P_max, int binned,
               unsigned long long beta_ppm, int budget, int32_t* __restrict__ src_map,
               int32_t* __restrict__ meta, int32_t* __restrict__ nout, int32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* keys = reinterpret_cast<uint64_t*>(smem_raw);
    int32_t* flag = reinterpret_cast<int32_t*>(keys + P_max);      // [cap]
    uint64_t* keys2 = reinterpret_cast<uint64_t*>(flag + ((cap + 1) & ~1));            // [P_max], binned only
    int32_t* bins = reinterpret_cast<int32_t*>(keys2 + P_max);                         // [2 * kPlanBins + 1]
    __shared__ int scan_scratch[33];
    __shared__ long long scan_ll[33];
    __shared__ unsigned long long s_thr;
    __shared__ int s_below, s_first_drop;

    pdl_enter();
    const int g = blockIdx.x, b = blockIdx.y;
    const int m_idx = b * Hkv + g;
    const int ln = len[m_idx];
    int32_t* src = src_map + (int64_t)m_idx * cap;
    float* acc = acc_score + (int64_t)m_idx * cap;
    if (ln < 0 || ln > cap) {
        if (threadIdx.x == 0) {
            if (dev_status) atomicOr(dev_status, LVLM_DEV_BOUNDS);
            meta[m_idx] = 0; nout[m_idx] = 0;           // nothing moves, length left as it is
        }
        return;
    }
    int lo = e_lo ? e_lo[b] : 0;
    int hi = e_hi ? e_hi[b] : ln;
    hi = min(hi, ln - recent);
    lo = min(max(lo, 0), ln);
    hi = max(hi, lo);
    const int m = hi - lo;
    int P = 2;
    while (P < m) P <<= 1;

    bool nonfinite = false;
    if (threadIdx.x == 0) { s_below = 0; s_first_drop = m; }
    for (int j = threadIdx.x; j < P; j += blockDim.x) {
        uint64_t key = ~0ull;
        if (j < m) key = ((uint64_t)desc_key(acc[lo + j], &nonfinite) << 32) | (uint32_t)j;
        keys[j] = key;
    }
    if (nonfinite && dev_status) atomicOr(dev_status, LVLM_DEV_NONFINITE);
    __syncthreads();
    if (binned && m >= kPlanBinFrom) {
        block_order_by_bins(keys, keys2, m, flag, bins, scan_scratch);
        keys = keys2;
    } else {
        block_bitonic_sort(keys, P);
    }

    // ---- how many entries of E reach the threshold ---------------------------------------
    int k_beta = m;
    if (beta_ppm < 1000000ull && m > 0) {
        const int per = (m + blockDim.x - 1) / blockDim.x;
        const int p0 = min(m, (int)threadIdx.x * per), p1 = min(m, p0 + per);
        long long part = 0;
        for (int p = p0; p < p1; ++p) part += score_units(acc[lo + (int)(uint32_t)keys[p]]);
        long long total;
        long long cum = block_exclusive_scan_ll(part, scan_ll, &total);
        if (threadIdx.x == 0) s_thr = ceil_muldiv(beta_ppm, (unsigned long long)total, 1000000ull);
        __syncthreads();
        const unsigned long long thr = s_thr;
        int below = 0;                                   // prefixes whose sum is still short
        for (int p = p0; p < p1; ++p) {
            cum += score_units(acc[lo + (int)(uint32_t)keys[p]]);
            if ((unsigned long long)cum < thr) ++below;
        }
        below = warp_sum(below);
        if ((threadIdx.x & 31) == 0 && below) atomicAdd(&s_below, below);
        __syncthreads();
        k_beta = min(m, s_below + 1);
    }
    int kc = k_beta;
    if (budget > 0) kc = min(kc, budget - (ln - m));
    kc = min(max(kc, 0), m);

    for (int j = threadIdx.x; j < m; j += blockDim.x) flag[j] = 0;
    __syncthreads();
    for (int p = threadIdx.x; p < kc; p += blockDim.x) flag[(int)(uint32_t)keys[p]] = 1;
    __syncthreads();

    // ---- survivor map -----------------------------------------------------------------------
    {
        const int per = (m + blockDim.x - 1) / blockDim.x;
        const int j0 = min(m, (int)threadIdx.x * per), j1 = min(m, j0 + per);
        int cnt = 0, first_drop = m;
        for (int j = j0; j < j1; ++j) {
            if (flag[j]) ++cnt; else if (first_drop == m) first_drop = j;
        }
        int total;
        int off = block_exclusive_scan(cnt, scan_scratch, &total);
        if (first_drop < m) atomicMin(&s_first_drop, first_drop);
        for (int j = j0; j < j1; ++j)
            if (flag[j]) src[lo + off++] = lo + j;
    }
    const int new_len = lo + kc + (ln - hi);
    for (int o = threadIdx.x; o < new_len; o += blockDim.x) {
        if (o < lo) src[o] = o;
        else if (o >= lo + kc) src[o] = hi + (o - lo - kc);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        meta[m_idx] = kc < m ? lo + s_first_drop : new_len;
        nout[m_idx] = new_len;
        len[m_idx] = new_len;
    }
    // ---- per-entry arrays, in place, tiles in increasing order ---------------------------------
    const int start = kc < m ? lo + s_first_drop : new_len;
    int32_t* ps = pos ? pos + (int64_t)m_idx * cap : nullptr;
    for (int o0 = start; o0 < new_len; o0 += blockDim.x) {
        const int o = o0 + threadIdx.x;
        float a = 0.f; int pv = 0;
        __syncthreads();
        if (o < new_len) { const int s = src[o]; a = acc[s]; if (ps) pv = ps[s]; }
        __syncthreads();
        if (o < new_len) { acc[o] = a; if (ps) ps[o] = pv; }
    }
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_kv_compress(void* Kc, void* Vc, float* acc_score, int32_t* pos,
                                         int32_t* len, const int32_t* e_lo, const int32_t* e_hi,
                                         const lvlm_dims* d, float beta, int budget, void* ws,
                                         size_t ws_bytes, int32_t* dev_status, void* stream_) {
    using namespace lvlm;
    cudaStream_t stream = (cudaStream_t)stream_;
    KvLayout L;
    if (!Kc || !Vc || !acc_score || !len || !kv_layout(d, &L)) return LVLM_ERR_INVALID_ARG;
    if ((e_lo == nullptr) != (e_hi == nullptr)) return LVLM_ERR_INVALID_ARG;
    if (!(beta > 0.f) || beta > 1.f) return LVLM_ERR_INVALID_ARG;
    if (d->D != kHeadDim || d->cap > kMaxSortN) return LVLM_ERR_UNSUPPORTED;
    const int64_t kv_sh = d->kv_stride_h ? d->kv_stride_h : (int64_t)d->cap * d->D;
    const int64_t kv_sb = d->kv_stride_b ? d->kv_stride_b : (int64_t)d->Hkv * kv_sh;
    if (!aligned16(Kc) || !aligned16(Vc) || kv_sh % 8 || kv_sb % 8) return LVLM_ERR_ALIGNMENT;
    if (!ws || !aligned256(ws) || ws_bytes < L.total) return LVLM_ERR_WORKSPACE;
    char* wsb = static_cast<char*>(ws);
    int32_t* src_map = reinterpret_cast<int32_t*>(wsb + L.off_src);
    int32_t* meta = reinterpret_cast<int32_t*>(wsb + L.off_meta);
    int32_t* nout = reinterpret_cast<int32_t*>(wsb + L.off_nout);

    const unsigned long long beta_ppm = (unsigned long long)llrint((double)beta * 1.0e6);
    const int P_max = next_pow2(d->cap < 2 ? 2 : d->cap);
    int threads = P_max / 2;
    threads = threads < 64 ? 64 : (threads > 1024 ? 1024 : threads);
    const int binned = d->cap >= kPlanBinFrom && d->cap <= kPlanBinMaxCap;
    const size_t smem = (size_t)P_max * 8 + (size_t)((d->cap + 1) & ~1) * 4 +
                        (binned ? (size_t)P_max * 8 + (size_t)(2 * kPlanBins + 2) * 4 : 0);
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(kv_plan_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    {
        const lvlm_status st = launch_kernel(kv_plan_kernel, dim3(d->Hkv, d->B), dim3(threads), smem, stream, 1,
                                             acc_score, pos, len, e_lo, e_hi, d->Hkv, d->cap, d->recent, P_max, binned,
                                             beta_ppm, budget, src_map, meta, nout, dev_status);
        if (st != LVLM_OK) return st;
    }
    CompactJob j;
    j.base0 = Kc; j.base1 = Vc; j.stride_b = kv_sb * 2; j.stride_g = kv_sh * 2; j.B = d->B; j.G = d->Hkv;
    j.V = kHeadDim / 8; j.src_map = src_map; j.maps_per_g = d->Hkv; j.map_stride = d->cap;
    j.meta = meta; j.meta_stride = 1; j.nout = nout; j.N = d->cap;
    return launch_inplace_compact(j, stream);
}
