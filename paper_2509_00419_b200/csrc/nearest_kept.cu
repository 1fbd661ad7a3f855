// lvlm_merge_compact, mode LVLM_W_NEAREST_KEPT.  Not in the paper (which argues against
// similarity-based merging, Section 3.2.1, paragraph 3): every dropped image token is averaged
// into the kept image token whose hidden row has the highest cosine similarity with its own
// (lower kept index wins ties); masses make repeated merging a true mean.
//
// Launches, all on the caller's stream:
//   plan      one CTA per sequence: kept / dropped token lists, row maps, position ids, new length
//   rows      the streaming kernel of the hidden states: kept rows to their place in the output,
//             dropped rows side by side into scratch
//   norms     1 / |x_t| of every kept row
//   sim       dropped x kept similarity on the tensor cores (tcgen05, accumulators in TMEM, operands by
//             TMA), arg-max per dropped row in the epilogue, merged over column splits with atomicMax
//             on (similarity, ~index) keys
//   group     dropped tokens sorted by (kept token, own index) by rank counting -> segments
//   merge     every kept row becomes the mass-weighted mean of itself and its segment, in token order
//   K, V      the same mean per KV head into scratch, text rows shifted down in place, means stored
//   mass      token masses compacted in place
#include "common.cuh"
#include "compact.cuh"
#include "merge.cuh"
#include "sm100.cuh"
#include "rank_count.cuh"

namespace lvlm {

using namespace sm100;

struct NkLayout {
    int r, Nout, V;
    HiddenGrid grid;
    size_t off_assign, off_src, off_dst, off_kept, off_drop, off_inv, off_best, off_order, off_sorted, off_seg,
           off_meta, off_newmass, off_scratch, off_kvtmp, total;
};

static bool nk_layout(const lvlm_dims* d, NkLayout* L) {
    if (!d || d->B <= 0 || d->N <= 0 || d->n <= 0 || d->C <= 0 || d->C % 8 || d->i0 < 0 ||
        d->k < 0 || d->k > d->n || (int64_t)d->i0 + d->n > d->N)
        return false;
    const size_t B = d->B, k = d->k, r = d->n - d->k;
    L->r = (int)r;
    L->Nout = d->N - (int)r;
    L->V = d->C / 8;
    L->grid = hidden_grid(d);
    size_t off = 0;
    L->off_assign = off;  off = align_up(off + B * (r ? r : 1) * 4, 256);   // first: callers may read it
    L->off_src = off;     off = align_up(off + B * d->N * 4, 256);
    L->off_dst = off;     off = align_up(off + B * d->N * 4, 256);
    L->off_kept = off;    off = align_up(off + B * (k ? k : 1) * 4, 256);
    L->off_drop = off;    off = align_up(off + B * (r ? r : 1) * 4, 256);
    L->off_inv = off;     off = align_up(off + B * (k ? k : 1) * 4, 256);
    L->off_best = off;    off = align_up(off + B * (r ? r : 1) * 8, 256);
    L->off_order = off;   off = align_up(off + B * (r ? r : 1) * 4, 256);
    L->off_sorted = off;  off = align_up(off + B * (r ? r : 1) * 4, 256);
    L->off_seg = off;     off = align_up(off + B * (k + 1) * 4, 256);
    L->off_meta = off;    off = align_up(off + B * kMetaInts * 4, 256);
    L->off_newmass = off; off = align_up(off + B * (k ? k : 1) * 4, 256);
    L->off_scratch = off; off = align_up(off + B * (r ? r : 1) * (size_t)d->C * 2, 256);
    L->off_kvtmp = off;
    if (d->Hkv > 0) off = align_up(off + B * d->Hkv * 2 * (k ? k : 1) * (size_t)kHeadDim * 2, 256);
    L->total = off;
    return true;
}

size_t nearest_kept_workspace(const lvlm_dims* d) {
    NkLayout L;
    return nk_layout(d, &L) ? L.total : 0;
}

// ---- plan ------------------------------------------------------------------------------------------
// One CTA per sequence.  kept[q] / drop[q]: image-token indices in ascending order.
// dst[i]: output row of input row i, or -2-q for the q-th dropped token.  src[o]: input row of
// output row o.  Position ids are compacted in place (tile by tile, sources lie at or after
// their destination).
__global__ void __launch_bounds__(1024)
nk_plan_kernel(const int32_t* __restrict__ rank, int32_t* pos_ids, int N, int i0, int n, int k,
               int32_t* __restrict__ src_map, int32_t* __restrict__ dst_map, int32_t* __restrict__ kept,
               int32_t* __restrict__ drop, unsigned long long* __restrict__ best, int32_t* __restrict__ meta,
               int32_t* new_len, int32_t* dev_status) {
    __shared__ int scan_scratch[33];
    pdl_enter();
    const int b = blockIdx.x, r = n - k, Nout = N - r;
    const int32_t* rk = rank + (int64_t)b * n;
    int32_t* src = src_map + (int64_t)b * N;
    int32_t* dst = dst_map + (int64_t)b * N;
    const int per = (n + blockDim.x - 1) / blockDim.x;
    const int j0 = min(n, (int)threadIdx.x * per), j1 = min(n, j0 + per);
    int cnt = 0;
    bool bad = false;
    for (int j = j0; j < j1; ++j) {
        const int rj = rk[j];
        if (rj < 0 || rj >= n) bad = true;
        cnt += rj < k;
    }
    int total;
    int kq = block_exclusive_scan(cnt, scan_scratch, &total);      // kept tokens before j0
    if (total != k) bad = true;
    int dq = j0 - kq;                                              // dropped tokens before j0
    for (int j = j0; j < j1; ++j) {
        if (rk[j] < k) {
            if (kq < k) { kept[(int64_t)b * k + kq] = j; src[i0 + kq] = i0 + j; dst[i0 + j] = i0 + kq; }
            else dst[i0 + j] = -2 - min(dq, max(r - 1, 0));
            ++kq;
        } else {
            if (dq < r) { drop[(int64_t)b * r + dq] = j; best[(int64_t)b * r + dq] = 0ull; dst[i0 + j] = -2 - dq; }
            else dst[i0 + j] = i0;                                 // inconsistent rank: flagged below
            ++dq;
        }
    }
    for (int o = threadIdx.x; o < Nout; o += blockDim.x) {
        if (o < i0) { src[o] = o; dst[o] = o; }
        else if (o >= i0 + k) { src[o] = o + r; dst[o + r] = o; }
    }
    if (bad && dev_status) atomicOr(dev_status, LVLM_DEV_BOUNDS);
    __syncthreads();
    if (threadIdx.x == 0) {
        meta[b * kMetaInts + 0] = i0;                               // first row of K, V that changes
        meta[b * kMetaInts + 1] = 0;
        if (new_len) new_len[b] = Nout;
    }
    if (pos_ids) {
        int32_t* pid = pos_ids + (int64_t)b * N;
        for (int o0 = 0; o0 < Nout; o0 += blockDim.x) {
            const int o = o0 + threadIdx.x;
            int val = 0;
            __syncthreads();
            if (o < Nout) val = pid[src[o]];
            __syncthreads();
            if (o < Nout) pid[o] = val;
        }
    }
}

// ---- norms -----------------------------------------------------------------------------------------
// One warp per kept row of the output: 1 / |x| in fp32 (1 for a zero row), fixed summation order.
__global__ void __launch_bounds__(256)
nk_norm_kernel(const uint4* __restrict__ out, int64_t out_stride_b, int V, int i0, int k,
               float* __restrict__ inv_norm) {
    pdl_enter();
    const int b = blockIdx.y, lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= k) return;
    const uint4* row = out + (int64_t)b * out_stride_b + (int64_t)(i0 + t) * V;
    float s = 0.f;
    for (int c = lane; c < V; c += 32) {
        const uint4 x = __ldg(row + c);
        const float e0 = bf16_lo(x.x), e1 = bf16_hi(x.x), e2 = bf16_lo(x.y), e3 = bf16_hi(x.y);
        const float e4 = bf16_lo(x.z), e5 = bf16_hi(x.z), e6 = bf16_lo(x.w), e7 = bf16_hi(x.w);
        s += (e0 * e0 + e1 * e1) + (e2 * e2 + e3 * e3) + (e4 * e4 + e5 * e5) + (e6 * e6 + e7 * e7);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if (lane == 0) inv_norm[(int64_t)b * k + t] = s > 0.f ? rsqrtf(s) : 1.f;
}

// ---- group -----------------------------------------------------------------------------------------
// Dropped tokens sorted by (kept token they go to, own order), by counting ranks: grid (blocks of 256
// dropped tokens, S, B), clusters (1, S, 1).  Writes the assignment, the sorted order and the kept
// token at every place of that order; a second kernel finds where every kept token's segment starts.
__global__ void __launch_bounds__(kRankThreads)
nk_group_kernel(const unsigned long long* __restrict__ best, int r, int k, int S, int slice_len, int jt,
                int32_t* __restrict__ assign, int32_t* __restrict__ order, int32_t* __restrict__ sorted_t) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_cnt[kRankMaxJT * kRankThreads];
    pdl_enter();
    const int b = blockIdx.z;
    const unsigned long long* bb = best + (int64_t)b * r;
    auto key_of = [&](int q) {
        const uint32_t t = 0xFFFFFFFFu - (uint32_t)(bb[q] & 0xFFFFFFFFull);
        return ((uint64_t)(t < (uint32_t)k ? t : 0u) << 32) | (uint32_t)q;     // nothing won: kept token 0
    };
    int p[kRankMaxJT];
    if (rank_by_counting(key_of, r, S, slice_len, jt, reinterpret_cast<uint64_t*>(smem_raw), s_cnt, p)) {
#pragma unroll
        for (int u = 0; u < kRankMaxJT; ++u) {
            const int q = rank_key_index(jt, u);
            if (u < jt && q < r) {
                const int t = (int)(key_of(q) >> 32);
                assign[(int64_t)b * r + q] = t;
                order[(int64_t)b * r + p[u]] = q;
                sorted_t[(int64_t)b * r + p[u]] = t;
            }
        }
    }
}

// seg[t] = first place of the sorted order whose kept token is >= t (t = 0..k).
__global__ void __launch_bounds__(256)
nk_seg_kernel(const int32_t* __restrict__ sorted_t, int r, int k, int32_t* __restrict__ seg) {
    pdl_enter();
    const int b = blockIdx.y, t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t > k) return;
    const int32_t* st = sorted_t + (int64_t)b * r;
    int lo = 0, hi = r;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (st[mid] < t) lo = mid + 1; else hi = mid;
    }
    seg[(int64_t)b * (k + 1) + t] = lo;
}

// ---- merge of the hidden rows ------------------------------------------------------------------------
// grid (CTAs per sequence, B); a CTA takes kept rows cta, cta + grid.x, ... (segments differ in
// length, striding evens them out).  Thread = 16-byte column group (+256 ...).  Row t of the output
// already holds x_t; its segment's rows come from scratch, four in flight, added in token order.
constexpr int kNkThreads = 256;

template <int CH>
__global__ void __launch_bounds__(kNkThreads)
nk_merge_kernel(uint4* __restrict__ out, int64_t out_stride_b, const uint4* __restrict__ scratch,
                int64_t scr_stride_b, int V, int N, int i0, int k, int r,
                const int32_t* __restrict__ kept, const int32_t* __restrict__ drop,
                const int32_t* __restrict__ order, const int32_t* __restrict__ seg,
                const float* __restrict__ mass, float* __restrict__ newmass) {
    pdl_enter();
    const int b = blockIdx.y, tid = threadIdx.x;
    uint4* orow = out + (int64_t)b * out_stride_b + (int64_t)i0 * V;
    const uint4* srow = scratch + (int64_t)b * scr_stride_b;
    const int32_t* ord = order + (int64_t)b * r;
    const int32_t* dr = drop + (int64_t)b * r;
    const float* ms = mass ? mass + (int64_t)b * N + i0 : nullptr;
    for (int t = blockIdx.x; t < k; t += gridDim.x) {
        const int p0 = seg[(int64_t)b * (k + 1) + t], p1 = seg[(int64_t)b * (k + 1) + t + 1];
        const float mt = ms ? ms[kept[(int64_t)b * k + t]] : 1.f;
        float den = mt;
        float acc[CH][8];
#pragma unroll
        for (int ci = 0; ci < CH; ++ci) {
            const int c = tid + ci * kNkThreads;
            const uint4 x = c < V ? orow[(int64_t)t * V + c] : make_uint4(0, 0, 0, 0);
            acc[ci][0] = mt * bf16_lo(x.x); acc[ci][1] = mt * bf16_hi(x.x);
            acc[ci][2] = mt * bf16_lo(x.y); acc[ci][3] = mt * bf16_hi(x.y);
            acc[ci][4] = mt * bf16_lo(x.z); acc[ci][5] = mt * bf16_hi(x.z);
            acc[ci][6] = mt * bf16_lo(x.w); acc[ci][7] = mt * bf16_hi(x.w);
        }
        for (int pb = p0; pb < p1; pb += 4) {
            float md[4];
            uint4 x[4][CH];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int p = pb + u;
                const int q = p < p1 ? ord[p] : 0;
                md[u] = p < p1 ? (ms ? ms[dr[q]] : 1.f) : 0.f;
#pragma unroll
                for (int ci = 0; ci < CH; ++ci) {
                    const int c = tid + ci * kNkThreads;
                    x[u][ci] = (p < p1 && c < V) ? __ldg(srow + (int64_t)q * V + c) : make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (pb + u < p1) {
                    den += md[u];
#pragma unroll
                    for (int ci = 0; ci < CH; ++ci) {
                        const uint4 xv = x[u][ci];
                        acc[ci][0] = fmaf(md[u], bf16_lo(xv.x), acc[ci][0]); acc[ci][1] = fmaf(md[u], bf16_hi(xv.x), acc[ci][1]);
                        acc[ci][2] = fmaf(md[u], bf16_lo(xv.y), acc[ci][2]); acc[ci][3] = fmaf(md[u], bf16_hi(xv.y), acc[ci][3]);
                        acc[ci][4] = fmaf(md[u], bf16_lo(xv.z), acc[ci][4]); acc[ci][5] = fmaf(md[u], bf16_hi(xv.z), acc[ci][5]);
                        acc[ci][6] = fmaf(md[u], bf16_lo(xv.w), acc[ci][6]); acc[ci][7] = fmaf(md[u], bf16_hi(xv.w), acc[ci][7]);
                    }
                }
            }
        }
        if (p1 > p0) {                                      // a row nothing was merged into stays as it is
            const float inv = 1.0f / den;
#pragma unroll
            for (int ci = 0; ci < CH; ++ci) {
                const int c = tid + ci * kNkThreads;
                if (c < V) {
                    uint4 o;
                    o.x = pack_bf16(acc[ci][0] * inv, acc[ci][1] * inv); o.y = pack_bf16(acc[ci][2] * inv, acc[ci][3] * inv);
                    o.z = pack_bf16(acc[ci][4] * inv, acc[ci][5] * inv); o.w = pack_bf16(acc[ci][6] * inv, acc[ci][7] * inv);
                    orow[(int64_t)t * V + c] = o;
                }
            }
        }
        if (tid == 0) newmass[(int64_t)b * k + t] = den;
    }
}

// ---- K and V ---------------------------------------------------------------------------------------------
// The same mean per (sequence, KV head, tensor), read from the cache as it stands before compaction and
// parked in scratch: 16 threads per 256-byte row, 16 kept rows per CTA.
__global__ void __launch_bounds__(kNkThreads)
nk_kv_merge_kernel(const uint4* __restrict__ Kc, const uint4* __restrict__ Vc, int64_t kv_sb, int64_t kv_sh,
                   int Hkv, int N, int i0, int k, int r, const int32_t* __restrict__ kept,
                   const int32_t* __restrict__ drop, const int32_t* __restrict__ order,
                   const int32_t* __restrict__ seg, const float* __restrict__ mass, uint4* __restrict__ kvtmp) {
    pdl_enter();
    const int b = blockIdx.z, g = blockIdx.y >> 1, which = blockIdx.y & 1;
    const int c = threadIdx.x & 15, t = blockIdx.x * 16 + (threadIdx.x >> 4);
    if (t >= k) return;
    const uint4* rows = (which ? Vc : Kc) + (int64_t)b * kv_sb + (int64_t)g * kv_sh + (int64_t)i0 * 16;
    const float* ms = mass ? mass + (int64_t)b * N + i0 : nullptr;
    const int32_t* ord = order + (int64_t)b * r;
    const int32_t* dr = drop + (int64_t)b * r;
    const int jt = kept[(int64_t)b * k + t];
    const int p0 = seg[(int64_t)b * (k + 1) + t], p1 = seg[(int64_t)b * (k + 1) + t + 1];
    const float mt = ms ? ms[jt] : 1.f;
    float den = mt, acc[8];
    {
        const uint4 x = rows[(int64_t)jt * 16 + c];
        acc[0] = mt * bf16_lo(x.x); acc[1] = mt * bf16_hi(x.x); acc[2] = mt * bf16_lo(x.y); acc[3] = mt * bf16_hi(x.y);
        acc[4] = mt * bf16_lo(x.z); acc[5] = mt * bf16_hi(x.z); acc[6] = mt * bf16_lo(x.w); acc[7] = mt * bf16_hi(x.w);
    }
    for (int pb = p0; pb < p1; pb += 4) {
        float md[4];
        uint4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int p = pb + u;
            const int jd = p < p1 ? dr[ord[p]] : 0;
            md[u] = p < p1 ? (ms ? ms[jd] : 1.f) : 0.f;
            x[u] = p < p1 ? rows[(int64_t)jd * 16 + c] : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (pb + u < p1) {
                den += md[u];
                acc[0] = fmaf(md[u], bf16_lo(x[u].x), acc[0]); acc[1] = fmaf(md[u], bf16_hi(x[u].x), acc[1]);
                acc[2] = fmaf(md[u], bf16_lo(x[u].y), acc[2]); acc[3] = fmaf(md[u], bf16_hi(x[u].y), acc[3]);
                acc[4] = fmaf(md[u], bf16_lo(x[u].z), acc[4]); acc[5] = fmaf(md[u], bf16_hi(x[u].z), acc[5]);
                acc[6] = fmaf(md[u], bf16_lo(x[u].w), acc[6]); acc[7] = fmaf(md[u], bf16_hi(x[u].w), acc[7]);
            }
        }
    }
    const float inv = 1.0f / den;
    uint4 o;
    if (p1 > p0) {
        o.x = pack_bf16(acc[0] * inv, acc[1] * inv); o.y = pack_bf16(acc[2] * inv, acc[3] * inv);
        o.z = pack_bf16(acc[4] * inv, acc[5] * inv); o.w = pack_bf16(acc[6] * inv, acc[7] * inv);
    } else {
        o = rows[(int64_t)jt * 16 + c];                           // nothing merged in: the row as it is
    }
    kvtmp[((((int64_t)b * Hkv + g) * 2 + which) * k + t) * 16 + c] = o;
}

__global__ void __launch_bounds__(kNkThreads)
nk_kv_store_kernel(uint4* __restrict__ Kc, uint4* __restrict__ Vc, int64_t kv_sb, int64_t kv_sh, int Hkv,
                   int i0, int k, const uint4* __restrict__ kvtmp) {
    pdl_enter();
    const int b = blockIdx.z, g = blockIdx.y >> 1, which = blockIdx.y & 1;
    const int c = threadIdx.x & 15, t = blockIdx.x * 16 + (threadIdx.x >> 4);
    if (t >= k) return;
    uint4* rows = (which ? Vc : Kc) + (int64_t)b * kv_sb + (int64_t)g * kv_sh + (int64_t)i0 * 16;
    rows[(int64_t)t * 16 + c] = kvtmp[((((int64_t)b * Hkv + g) * 2 + which) * k + t) * 16 + c];
}

// Token masses, in place: the kept tokens take their new mass, the rows behind the image move up.
__global__ void __launch_bounds__(1024)
nk_mass_kernel(float* mass, int N, int i0, int k, int r, const float* __restrict__ newmass) {
    pdl_enter();
    const int b = blockIdx.x, Nout = N - r;
    float* m = mass + (int64_t)b * N;
    for (int o0 = i0; o0 < Nout; o0 += blockDim.x) {
        const int o = o0 + threadIdx.x;
        float val = 0.f;
        __syncthreads();
        if (o < Nout) val = o < i0 + k ? newmass[(int64_t)b * k + (o - i0)] : m[o + r];
        __syncthreads();
        if (o < Nout) m[o] = val;
    }
}

// ---- similarity on the tensor cores --------------------------------------------------------------------
// S = X_dropped X_kept^T, 128 dropped rows x 256 kept columns per accumulator, K = channels in chunks
// of 64.  grid (row tiles, column splits, B).  Warp 0 feeds a ring of shared-memory stages by TMA,
// warp 1 issues the MMAs into two TMEM accumulators in turn, eight epilogue warps scale the columns by
// 1/|x_t| and keep the best (value, kept index) of their row while the next accumulator fills.
constexpr int kSimM = 128, kSimN = 256, kSimK = 64, kSimStages = 4;
constexpr int kSimABytes = kSimM * kSimK * 2, kSimBBytes = kSimN * kSimK * 2;
constexpr int kSimStageBytes = kSimABytes + kSimBBytes;
constexpr int kSimThreads = 320, kSimEpi = 256;
constexpr uint32_t kSimTmemCols = 512;

struct SimArgs {
    int r, k, nkc, nct, cps;
    const float* inv_norm;          // [B][k]
    unsigned long long* best;       // [B][r] (orderable similarity << 32) | ~kept index, zero before
    int32_t* dev_status;
};

struct SimSmem {
    uint64_t full[kSimStages], empty[kSimStages], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort;
    float inv_s[8][2][128];         // per epilogue warp and accumulator: 1/|x_t| of its 128 columns
    float xv[kSimM];                // upper column half's best, handed to the lower half
    int xt[kSimM];
};

__device__ __forceinline__ bool sim_wait(uint64_t* bar, uint32_t parity, SimSmem* sm, int32_t* dev_status) {
    if (sm->abort) return false;
    if (mbar_wait(bar, parity)) return true;
    sm->abort = 1;
    if (dev_status) atomicOr(dev_status, LVLM_DEV_TIMEOUT);
    return false;
}

__global__ void __launch_bounds__(kSimThreads, 1)
nk_sim_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap, const SimArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    SimSmem* sm = reinterpret_cast<SimSmem*>(base + kSimStageBytes * kSimStages);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rt = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
    const int ct0 = split * a.cps, ct1 = min(a.nct, ct0 + a.cps);
    const int ntile = max(0, ct1 - ct0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSimStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sm->tmem_full[s], 1); mbar_init(&sm->tmem_empty[s], kSimEpi); }
        sm->abort = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&amap);
        prefetch_tmap(&bmap);
    }
    if (warp == 1) tmem_alloc(&sm->tmem_base, kSimTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    pdl_enter();

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            for (int j = 0; j < ntile; ++j) {
                for (int kc = 0; kc < a.nkc; ++kc, ++it) {
                    const int st = it % kSimStages;
                    if (it >= kSimStages && !sim_wait(&sm->empty[st], ((it / kSimStages) - 1) & 1, sm, a.dev_status)) { j = ntile; break; }
                    unsigned char* dst = base + st * kSimStageBytes;
                    mbar_arrive_expect_tx(&sm->full[st], kSimStageBytes);
                    tma_load_3d(dst, &amap, &sm->full[st], kc * kSimK, rt * kSimM, b);
                    tma_load_3d(dst + kSimABytes, &bmap, &sm->full[st], kc * kSimK, (ct0 + j) * kSimN, b);
                }
            }
        }
    } else if (warp == 1) {
        // all lanes run the loop (uniform operands), one elected lane issues
        {
            constexpr uint32_t idesc = idesc_bf16_f32(kSimM, kSimN);
            int it = 0;
            bool ok = true;
            for (int j = 0; ok && j < ntile; ++j) {
                const int buf = j & 1;
                if (j >= 2) ok = __all_sync(0xFFFFFFFFu, sim_wait(&sm->tmem_empty[buf], ((j / 2) - 1) & 1, sm, a.dev_status));
                for (int kc = 0; ok && kc < a.nkc; ++kc, ++it) {
                    const int st = it % kSimStages;
                    const uint32_t a_addr = smem_u32(base + st * kSimStageBytes);
                    const uint32_t b_addr = a_addr + kSimABytes;
                    const uint32_t d_tmem = tmem_base + buf * kSimN;
                    uint64_t ad[4], bd[4];
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) { ad[kk] = smem_desc_sw128(a_addr + kk * 32); bd[kk] = smem_desc_sw128(b_addr + kk * 32); }
                    ok = __all_sync(0xFFFFFFFFu, sim_wait(&sm->full[st], (it / kSimStages) & 1, sm, a.dev_status));
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_bf16_ss(d_tmem, ad[kk], bd[kk], idesc, (kc > 0 || kk > 0) ? 1u : 0u);
                        mma_commit(&sm->empty[st]);
                    }
                    __syncwarp();
                }
                if (ok && elect_one()) mma_commit(&sm->tmem_full[buf]);
                __syncwarp();
            }
        }
    } else {
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const float* inv = a.inv_norm + (int64_t)b * a.k;
        float best_v = -INFINITY;
        int best_t = -1;
        float inv_next[4];
        auto fetch_inv = [&](int j) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int t = (ct0 + j) * kSimN + half * 128 + u * 32 + lane;
                inv_next[u] = t < a.k ? __ldg(inv + t) : 0.f;
            }
        };
        if (ntile > 0) fetch_inv(0);
        for (int j = 0; j < ntile; ++j) {
            const int buf = j & 1;
#pragma unroll
            for (int u = 0; u < 4; ++u) sm->inv_s[warp - 2][buf][u * 32 + lane] = inv_next[u];
            if (j + 1 < ntile) fetch_inv(j + 1);
            __syncwarp();
            if (!sim_wait(&sm->tmem_full[buf], (j / 2) & 1, sm, a.dev_status)) break;
            tc_fence_after();
#pragma unroll 1
            for (int c4 = 0; c4 < 4; ++c4) {
                float v[32];
                tmem_ld32(lane_addr + buf * kSimN + half * 128 + c4 * 32, v);
                tmem_ld_wait();
                const int tb = (ct0 + j) * kSimN + half * 128 + c4 * 32;
                const float* is = &sm->inv_s[warp - 2][buf][c4 * 32];
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const float val = v[c] * is[c];
                    if (tb + c < a.k && val > best_v) { best_v = val; best_t = tb + c; }
                }
            }
            tc_fence_before();
            mbar_arrive(&sm->tmem_empty[buf]);
        }
        // the two column halves of a row meet in shared memory (on equal similarity the lower kept index
        // wins, whichever half and column tile it sits in); every epilogue thread comes here, also after a timeout
        if (half == 1) { sm->xv[row] = best_v; sm->xt[row] = best_t; }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (half == 0) {
            const float ov = sm->xv[row];
            const int ot = sm->xt[row];
            if (ot >= 0 && (best_t < 0 || ov > best_v || (ov == best_v && ot < best_t))) { best_v = ov; best_t = ot; }
            const int q = rt * kSimM + row;
            if (!sm->abort && q < a.r && best_t >= 0) {
                uint32_t u = __float_as_uint(best_v);
                u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);         // ascending in the value
                const unsigned long long key = ((unsigned long long)u << 32) | (0xFFFFFFFFu - (uint32_t)best_t);
                atomicMax(a.best + (int64_t)b * a.r + q, key);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (sm->abort) {
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kSimTmemCols);
    }
}

template <int CH>
static lvlm_status launch_nk_merge(void* out, int64_t out_sb, const void* scratch, int64_t scr_sb, const lvlm_dims* d,
                                   const NkLayout& L, const int32_t* kept, const int32_t* drop, const int32_t* order,
                                   const int32_t* seg, const float* mass, float* newmass, cudaStream_t stream) {
    int ctas = (4 * 148) / d->B;
    ctas = ctas < 1 ? 1 : (ctas > d->k ? d->k : ctas);
    return launch_kernel(nk_merge_kernel<CH>, dim3(ctas, d->B), dim3(kNkThreads), 0, stream, 1,
                         static_cast<uint4*>(out), out_sb / 8, static_cast<const uint4*>(scratch), scr_sb / 8, L.V,
                         d->N, d->i0, d->k, L.r, kept, drop, order, seg, mass, newmass);
}

lvlm_status launch_nearest_kept(const void* hidden, void* hidden_out, void* Kc, void* Vc, int32_t* pos_ids,
                                const int32_t* rank, const lvlm_dims* d, float* mass, int32_t* new_len,
                                void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t stream) {
    NkLayout L;
    if (!nk_layout(d, &L) || d->k < 1) return LVLM_ERR_INVALID_ARG;
    if (!hidden_out || hidden_out == hidden) return LVLM_ERR_UNSUPPORTED;     // out of place only
    if (L.r > kRankMaxKeys) return LVLM_ERR_UNSUPPORTED;       // the slices of the keys have to fit in shared memory
    if (!ws || !aligned256(ws) || ws_bytes < L.total) return LVLM_ERR_WORKSPACE;
    const int64_t hid_sb = d->hid_stride_b ? d->hid_stride_b : (int64_t)d->N * d->C;
    const int64_t out_sb = d->out_stride_b ? d->out_stride_b : (int64_t)L.Nout * d->C;
    const int64_t kv_sh = d->kv_stride_h ? d->kv_stride_h : (int64_t)d->cap * d->D;
    const int64_t kv_sb = d->kv_stride_b ? d->kv_stride_b : (int64_t)d->Hkv * kv_sh;
    const int64_t scr_sb = (int64_t)L.r * d->C;
    char* wsb = static_cast<char*>(ws);
    int32_t* assign = reinterpret_cast<int32_t*>(wsb + L.off_assign);
    int32_t* src_map = reinterpret_cast<int32_t*>(wsb + L.off_src);
    int32_t* dst_map = reinterpret_cast<int32_t*>(wsb + L.off_dst);
    int32_t* kept = reinterpret_cast<int32_t*>(wsb + L.off_kept);
    int32_t* drop = reinterpret_cast<int32_t*>(wsb + L.off_drop);
    float* inv_norm = reinterpret_cast<float*>(wsb + L.off_inv);
    unsigned long long* best = reinterpret_cast<unsigned long long*>(wsb + L.off_best);
    int32_t* order = reinterpret_cast<int32_t*>(wsb + L.off_order);
    int32_t* sorted_t = reinterpret_cast<int32_t*>(wsb + L.off_sorted);
    int32_t* seg = reinterpret_cast<int32_t*>(wsb + L.off_seg);
    int32_t* meta = reinterpret_cast<int32_t*>(wsb + L.off_meta);
    float* newmass = reinterpret_cast<float*>(wsb + L.off_newmass);
    void* scratch = wsb + L.off_scratch;
    uint4* kvtmp = reinterpret_cast<uint4*>(wsb + L.off_kvtmp);

    lvlm_status st;
    const int plan_threads = d->n >= 1024 ? 1024 : (d->n <= 128 ? 128 : ((d->n + 31) / 32) * 32);
    st = launch_kernel(nk_plan_kernel, dim3(d->B), dim3(plan_threads), 0, stream, 1, rank, pos_ids, d->N, d->i0,
                       d->n, d->k, src_map, dst_map, kept, drop, best, meta, new_len, dev_status);
    if (st != LVLM_OK) return st;
    st = launch_hidden_rows(hidden, hidden_out, hid_sb, out_sb, d, L.grid, dst_map, nullptr, meta, nullptr,
                            scratch, scr_sb, stream);
    if (st != LVLM_OK) return st;
    st = launch_kernel(nk_norm_kernel, dim3((d->k + 7) / 8, d->B), dim3(256), 0, stream, 1,
                       static_cast<const uint4*>(hidden_out), out_sb / 8, L.V, d->i0, d->k, inv_norm);
    if (st != LVLM_OK) return st;
    {
        CUtensorMap amap, bmap;
        const uint64_t adims[3] = {(uint64_t)d->C, (uint64_t)L.r, (uint64_t)d->B};
        const uint64_t astr[2] = {(uint64_t)d->C * 2, (uint64_t)scr_sb * 2};
        const uint32_t abox[3] = {(uint32_t)kSimK, (uint32_t)kSimM, 1};
        if (!make_tmap_bf16(&amap, scratch, 3, adims, astr, abox)) return LVLM_ERR_CUDA;
        const uint64_t bdims[3] = {(uint64_t)d->C, (uint64_t)d->k, (uint64_t)d->B};
        const uint64_t bstr[2] = {(uint64_t)d->C * 2, (uint64_t)out_sb * 2};
        const uint32_t bbox[3] = {(uint32_t)kSimK, (uint32_t)kSimN, 1};
        const void* bbase = static_cast<const char*>(hidden_out) + (int64_t)d->i0 * d->C * 2;
        if (!make_tmap_bf16(&bmap, bbase, 3, bdims, bstr, bbox)) return LVLM_ERR_CUDA;
        SimArgs a;
        a.r = L.r; a.k = d->k; a.nkc = (d->C + kSimK - 1) / kSimK; a.nct = (d->k + kSimN - 1) / kSimN;
        const int row_tiles = (L.r + kSimM - 1) / kSimM;
        // column splits: one CTA per SM at a time, so the kernel takes waves x (column tiles per CTA + a
        // little for the set-up of a CTA); take the split with the smallest product
        int nsplit = 1;
        double best_est = 1e30;
        for (int ns = 1; ns <= a.nct; ++ns) {
            const int cps = (a.nct + ns - 1) / ns, used = (a.nct + cps - 1) / cps;
            const int64_t ctas = (int64_t)row_tiles * d->B * used;
            const double est = (double)((ctas + 147) / 148) * (cps + 0.25);
            if (est < best_est - 1e-9) { best_est = est; nsplit = used; a.cps = cps; }
        }
        a.inv_norm = inv_norm; a.best = best; a.dev_status = dev_status;
        const size_t smem = 1024 + (size_t)kSimStageBytes * kSimStages + sizeof(SimSmem);
        LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(nk_sim_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem));
        st = launch_kernel(nk_sim_kernel, dim3(row_tiles, nsplit, d->B), dim3(kSimThreads), smem, stream, 1,
                           amap, bmap, a);
        if (st != LVLM_OK) return st;
    }
    {
        int S, slice_len, jt;
        rank_shape(L.r, d->B, &S, &slice_len, &jt);
        LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(nk_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 kMaxDynSmem));
        st = launch_kernel_cluster(nk_group_kernel, dim3((L.r + kRankThreads * jt - 1) / (kRankThreads * jt), S, d->B),
                                   dim3(kRankThreads), rank_smem_bytes(slice_len), stream, dim3(1, S, 1),
                                   best, L.r, d->k, S, slice_len, jt, assign, order, sorted_t);
        if (st != LVLM_OK) return st;
        st = launch_kernel(nk_seg_kernel, dim3((d->k + 1 + 255) / 256, d->B), dim3(256), 0, stream, 1,
                           sorted_t, L.r, d->k, seg);
        if (st != LVLM_OK) return st;
    }
    const int chunks = (L.V + kNkThreads - 1) / kNkThreads;
    switch (chunks) {
        case 1: st = launch_nk_merge<1>(hidden_out, out_sb, scratch, scr_sb, d, L, kept, drop, order, seg, mass, newmass, stream); break;
        case 2: st = launch_nk_merge<2>(hidden_out, out_sb, scratch, scr_sb, d, L, kept, drop, order, seg, mass, newmass, stream); break;
        case 3: st = launch_nk_merge<3>(hidden_out, out_sb, scratch, scr_sb, d, L, kept, drop, order, seg, mass, newmass, stream); break;
        case 4: st = launch_nk_merge<4>(hidden_out, out_sb, scratch, scr_sb, d, L, kept, drop, order, seg, mass, newmass, stream); break;
        default: return LVLM_ERR_UNSUPPORTED;
    }
    if (st != LVLM_OK) return st;
    if (Kc) {
        const dim3 grid((d->k + 15) / 16, d->Hkv * 2, d->B);
        st = launch_kernel(nk_kv_merge_kernel, grid, dim3(kNkThreads), 0, stream, 1, static_cast<const uint4*>(Kc),
                           static_cast<const uint4*>(Vc), kv_sb / 8, kv_sh / 8, d->Hkv, d->N, d->i0, d->k, L.r, kept,
                           drop, order, seg, mass, kvtmp);
        if (st != LVLM_OK) return st;
        CompactJob cj;
        cj.base0 = Kc; cj.base1 = Vc; cj.stride_b = kv_sb * 2; cj.stride_g = kv_sh * 2; cj.B = d->B; cj.G = d->Hkv;
        cj.V = kHeadDim / 8; cj.src_map = src_map; cj.map_stride = d->N; cj.meta = meta; cj.meta_stride = kMetaInts;
        cj.Nout = L.Nout; cj.N = d->N;
        st = launch_inplace_compact(cj, stream);
        if (st != LVLM_OK) return st;
        st = launch_kernel(nk_kv_store_kernel, grid, dim3(kNkThreads), 0, stream, 1, static_cast<uint4*>(Kc),
                           static_cast<uint4*>(Vc), kv_sb / 8, kv_sh / 8, d->Hkv, d->i0, d->k, kvtmp);
        if (st != LVLM_OK) return st;
    }
    if (mass)
        return launch_kernel(nk_mass_kernel, dim3(d->B), dim3(1024), 0, stream, 1, mass, d->N, d->i0, d->k, L.r,
                             newmass);
    return LVLM_OK;
}

}  // namespace lvlm
