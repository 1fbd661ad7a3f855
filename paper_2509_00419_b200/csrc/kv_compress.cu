// lvlm_kv_compress: per (sequence, KV head) eviction of low-score cache entries
// (Section 3.2.2, paragraph 2: sort the scores in descending order, keep the entries whose
// accumulated score reaches the threshold beta, discard the other image entries; Appendix A.2:
// beta = 0.995).  A plan kernel finds the entry at which the threshold (and the budget) is met,
// builds the survivor map and compacts the small per-entry arrays; the shared in-place compaction kernel
// then moves the K and V rows.
#include "common.cuh"
#include "compact.cuh"

namespace lvlm {

struct KvLayout { size_t off_src, off_meta, off_nout, off_acc, off_pos, total; };

static bool kv_layout(const lvlm_dims* d, KvLayout* L) {
    if (!d || d->B <= 0 || d->Hkv <= 0 || d->cap <= 0 || d->recent < 0) return false;
    size_t off = 0;
    const size_t heads = (size_t)d->B * d->Hkv;
    L->off_src = off;  off = align_up(off + heads * d->cap * 4, 256);
    L->off_meta = off; off = align_up(off + heads * 4, 256);
    L->off_nout = off; off = align_up(off + heads * 4, 256);
    L->off_acc = off;  off = align_up(off + heads * d->cap * 4, 256);     // compacted acc_score and pos, copied back
    L->off_pos = off;  off = align_up(off + heads * d->cap * 4, 256);     // by the kernel that moves the rows
    L->total = off;
    return true;
}

size_t kv_compress_workspace(const lvlm_dims* d) {
    KvLayout L;
    return kv_layout(d, &L) ? L.total : 0;
}

// Score in integer units of 2^-24 (negative and non-finite scores count as zero).
__device__ __forceinline__ long long score_units(float s) {
    if (!(s > 0.f) || (__float_as_uint(s) & 0x7F800000u) == 0x7F800000u) return 0;
    return __float2ll_rn(s * 16777216.0f);               // exact: a power of two (beyond 2^104 both saturate)
}

// ceil(a * b / c) for a, b < 2^63, c = 10^6, in 128-bit arithmetic.
__device__ __forceinline__ unsigned long long ceil_muldiv(unsigned long long a, unsigned long long b,
                                                          unsigned long long c) {
    unsigned long long hi = __umul64hi(a, b), lo = a * b;
    // long division of (hi:lo) by c, 64 steps; hi < c holds because a < c (beta < 1) ... not
    // assumed: reduce hi first.
    unsigned long long rem = hi % c;
    unsigned long long q = 0;
#pragma unroll 1
    for (int bit = 63; bit >= 0; --bit) {
        rem = (rem << 1) | ((lo >> bit) & 1ull);        // rem < 2c < 2^63, no overflow
        q <<= 1;
        if (rem >= c) { rem -= c; q |= 1ull; }
    }
    // the quotient's high word (hi / c) is zero whenever a <= c, which the caller guarantees
    return q + (rem != 0);
}

// Sums over the first `nwarp` warps of the block of a count and a 64-bit mass (one barrier: the scratch rows
// alternate with `turn`).
struct PlanScratch { int c[2][32]; unsigned long long m[2][32]; };
__device__ __forceinline__ void block_sum2(int* c, unsigned long long* ms, PlanScratch* sc, int turn, int nwarp) {
    int cc = *c;
    unsigned long long mm = *ms;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        cc += __shfl_xor_sync(0xFFFFFFFFu, cc, o);
        mm += __shfl_xor_sync(0xFFFFFFFFu, mm, o);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sc->c[turn][warp] = cc; sc->m[turn][warp] = mm; }
    asm volatile("bar.sync 1, %0;" ::"r"(nwarp * 32) : "memory");       // the warps that hold entries
    cc = 0; mm = 0;
    for (int wv = 0; wv < nwarp; ++wv) { cc += sc->c[turn][wv]; mm += sc->m[turn][wv]; }
    *c = cc; *ms = mm;
}

// One CTA per (sequence, KV head).  A thread holds KPT consecutive evictable entries as 64-bit keys (order-
// preserving image of the score above the index: ascending key = descending score, lower index first).  Nothing
// is sorted: the entry at which the accumulated score reaches the threshold, and the entry that closes the budget,
// are found by building the key bit by bit from the top - "do the entries up to this key reach the target?" is one
// sum over the block - and only over the bits in which the keys differ at all.  All sums are integers, so the
// result does not depend on the order of summation.
template <int KPT>
__global__ void __launch_bounds__(1024)
kv_plan_kernel(float* acc_score, int32_t* pos, int32_t* len, const int32_t* __restrict__ e_lo,
               const int32_t* __restrict__ e_hi, int Hkv, int cap, int recent, int min_m,
               unsigned long long beta_ppm, int budget, int32_t* __restrict__ src_map,
               int32_t* __restrict__ meta, int32_t* __restrict__ nout, float* __restrict__ acc_new,
               int32_t* __restrict__ pos_new, int32_t* dev_status) {
    __shared__ PlanScratch sc;
    __shared__ unsigned long long s_and[32], s_or[32];
    __shared__ int scan_scratch[33];
    __shared__ int s_first_drop;

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
    if (m < min_m) return;                               // a head this small was planned by the warp kernel
    // only the warps that hold entries stay: every barrier below counts them alone
    const int nwarp = max(1, (m + 32 * KPT - 1) / (32 * KPT)), nthr = nwarp * 32;
    if ((int)threadIdx.x >= nthr) return;
    auto sync_active = [&]() { asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory"); };
    if (threadIdx.x == 0) s_first_drop = m;
    // compacted acc_score and pos go beside the map; the kernel that moves the K and V rows copies them back
    float* an = acc_new + (int64_t)m_idx * cap;
    const int32_t* ps = pos ? pos + (int64_t)m_idx * cap : nullptr;
    int32_t* pn = pos_new + (int64_t)m_idx * cap;

    // ---- my keys -------------------------------------------------------------------------------------
    const int j0 = threadIdx.x * KPT;
    uint64_t key[KPT];
    unsigned long long un[KPT];                          // the scores in integer units
    bool nonfinite = false;
    uint64_t k_and = ~0ull, k_or = 0ull;
    unsigned long long total = 0;
    int turn = 0;
#pragma unroll
    for (int u = 0; u < KPT; ++u) {
        key[u] = ~0ull;                                  // past the end: above every real key
        un[u] = 0ull;
        if (j0 + u < m) {
            const float sv = acc[lo + j0 + u];
            key[u] = ((uint64_t)desc_key(sv, &nonfinite) << 32) | (uint32_t)(j0 + u);
            k_and &= key[u]; k_or |= key[u];
            un[u] = (unsigned long long)score_units(sv);
            total += un[u];
        }
    }
    if (nonfinite && dev_status) atomicOr(dev_status, LVLM_DEV_NONFINITE);
    {   // bits in which the keys differ, and the total score
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            k_and &= __shfl_xor_sync(0xFFFFFFFFu, k_and, o);
            k_or |= __shfl_xor_sync(0xFFFFFFFFu, k_or, o);
        }
        if ((threadIdx.x & 31) == 0) { s_and[threadIdx.x >> 5] = k_and; s_or[threadIdx.x >> 5] = k_or; }
        int dummy = 0;
        block_sum2(&dummy, &total, &sc, turn, nwarp); turn ^= 1;            // (its barrier also publishes s_and / s_or)
        k_and = ~0ull; k_or = 0ull;
        for (int wv = 0; wv < nwarp; ++wv) { k_and &= s_and[wv]; k_or |= s_or[wv]; }
    }
    const uint64_t diff = m > 0 ? (k_and ^ k_or) : 0ull;
    // Smallest key T such that the entries with key <= T hold at least `target` (their count, or their score when
    // by_mass).  The caller guarantees that all entries together reach the target.
    auto search = [&](unsigned long long target, bool by_mass) -> uint64_t {
        uint64_t ans = k_and;
        uint64_t todo = diff;
        while (todo) {
            const int bit = 63 - __clzll((long long)todo);
            todo &= ~(1ull << bit);
            const uint64_t cand = (ans & ~(1ull << bit)) | ((1ull << bit) - 1ull);
            int cnt = 0;
            unsigned long long ms = 0;
#pragma unroll
            for (int u = 0; u < KPT; ++u) {
                if (key[u] <= cand) { ++cnt; ms += un[u]; }
            }
            block_sum2(&cnt, &ms, &sc, turn, nwarp); turn ^= 1;
            const unsigned long long have = by_mass ? ms : (unsigned long long)cnt;
            if (have >= target) ans &= ~(1ull << bit); else ans |= 1ull << bit;
        }
        return ans;
    };
    auto count_upto = [&](uint64_t T) -> int {
        int cnt = 0;
        unsigned long long ms = 0;
#pragma unroll
        for (int u = 0; u < KPT; ++u) cnt += key[u] <= T;
        block_sum2(&cnt, &ms, &sc, turn, nwarp); turn ^= 1;
        return cnt;
    };

    // ---- how many entries of E reach the threshold, how many the budget allows ---------------------------
    int k_beta = m;
    uint64_t T = ~0ull;                                  // keys <= T survive
    bool have_T = false;
    if (beta_ppm < 1000000ull && m > 0) {
        const unsigned long long thr = ceil_muldiv(beta_ppm, total, 1000000ull);
        if (thr == 0) k_beta = 1;
        else {
            T = search(thr, true);
            k_beta = count_upto(T);
            have_T = true;
        }
    }
    int kc = k_beta;
    if (budget > 0) kc = min(kc, budget - (ln - m));
    kc = min(max(kc, 0), m);
    if (kc < m && kc > 0 && !(have_T && kc == k_beta)) T = search((unsigned long long)kc, false);

    // ---- survivor map: my entries are consecutive, so a scan of the counts gives their places ------------------
    {
        int cnt = 0, first_drop = m;
#pragma unroll
        for (int u = 0; u < KPT; ++u) {
            if (j0 + u < m) {
                const bool kept = kc >= m || (kc > 0 && key[u] <= T);
                if (kept) ++cnt; else if (first_drop == m) first_drop = j0 + u;
            }
        }
        // exclusive scan of the counts over the active warps
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) scan_scratch[warp] = incl;
        sync_active();
        int off = incl - cnt;
        for (int wv = 0; wv < warp; ++wv) off += scan_scratch[wv];
        if (first_drop < m) atomicMin(&s_first_drop, first_drop);
#pragma unroll
        for (int u = 0; u < KPT; ++u)
            if (j0 + u < m && (kc >= m || (kc > 0 && key[u] <= T))) {
                src[lo + off] = lo + j0 + u;
                an[lo + off] = acc[lo + j0 + u];
                if (ps) pn[lo + off] = ps[lo + j0 + u];
                ++off;
            }
    }
    const int new_len = lo + kc + (ln - hi);
    for (int o = threadIdx.x; o < new_len; o += nthr) {
        if (o < lo) src[o] = o;
        else if (o >= lo + kc) {
            const int sidx = hi + (o - lo - kc);
            src[o] = sidx;
            an[o] = acc[sidx];
            if (ps) pn[o] = ps[sidx];
        }
    }
    sync_active();
    if (threadIdx.x == 0) {
        meta[m_idx] = kc < m ? lo + s_first_drop : new_len;
        nout[m_idx] = new_len;
        len[m_idx] = new_len;
    }
}

// The same for caches of up to 2048 rows: one WARP per (sequence, KV head); lane l holds entries l, l + 32, ...
// (coalesced), every sum is a handful of shuffles and no barrier is needed, so an SM works on dozens of heads at
// once.  Only the 32-bit image of the score is searched: among entries of equal score the lower index comes first,
// so once the threshold score T is known, "the first `need` entries of score T" is a running count in index order
// and the index never has to enter the key.  The searches are loops over registers; the pass that writes the map
// is a loop over the entries that reads the scores again (they are in L1), which keeps the kernel's code short:
// a warp runs through it once, and straight-line code is fetched slower than it executes.
// MASS: the threshold beta is in use (without it only the budget's count search is compiled in).
__device__ __forceinline__ void plan_cp_async4(void* smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}

template <int KPL, bool MASS>
__global__ void __launch_bounds__(128)
kv_plan_warp_kernel(float* acc_score, int32_t* pos, int32_t* len, const int32_t* __restrict__ e_lo,
                    const int32_t* __restrict__ e_hi, int heads, int Hkv, int cap, int recent, int only_small,
                    unsigned long long beta_ppm, int budget, int32_t* __restrict__ src_map,
                    int32_t* __restrict__ meta, int32_t* __restrict__ nout, float* __restrict__ acc_new,
                    int32_t* __restrict__ pos_new, int32_t* dev_status) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int m_idx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (m_idx >= heads) return;
    const int b = m_idx / Hkv;
    const int ln = len[m_idx];
    int32_t* src = src_map + (int64_t)m_idx * cap;
    float* acc = acc_score + (int64_t)m_idx * cap;
    if (ln < 0 || ln > cap) {
        if (lane == 0) {
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
    if (only_small && m > 32 * KPL) return;              // too many entries for the registers: the CTA kernel plans it

    // The scores and the position ids of the evictable entries come to shared memory by asynchronous copies
    // (all of them in flight at once); the scores are turned into keys there, by a loop over the entries, and
    // then taken into registers.
    extern __shared__ __align__(16) uint32_t s_plan[];   // per warp: [KPL * 32] keys, [KPL * 32] position ids
    uint32_t* my_hk = s_plan + (threadIdx.x >> 5) * (2 * KPL * 32);
    uint32_t* my_pos = my_hk + KPL * 32;
    const int32_t* ps = pos ? pos + (int64_t)m_idx * cap : nullptr;
#pragma unroll 4
    for (int j = lane; j < m; j += 32) {
        plan_cp_async4(&my_hk[j], acc + lo + j);
        if (ps) plan_cp_async4(&my_pos[j], ps + lo + j);
    }
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
    __syncwarp();
    uint32_t k_and = ~0u, k_or = 0u;
    bool nonfinite = false;
#pragma unroll 4
    for (int j = lane; j < KPL * 32; j += 32) {
        uint32_t h = ~0u;                                // past the end: the top value
        if (j < m) { h = desc_key(__uint_as_float(my_hk[j]), &nonfinite); k_and &= h; k_or |= h; }
        my_hk[j] = h;
    }
    if (nonfinite && dev_status) atomicOr(dev_status, LVLM_DEV_NONFINITE);
    uint32_t hk[KPL];                                    // ascending = descending score
#pragma unroll
    for (int u = 0; u < KPL; ++u) hk[u] = my_hk[u * 32 + lane];       // (written by this very lane)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        k_and &= __shfl_xor_sync(0xFFFFFFFFu, k_and, o);
        k_or |= __shfl_xor_sync(0xFFFFFFFFu, k_or, o);
    }
    const uint32_t diff = m > 0 ? (k_and ^ k_or) : 0u;
    auto units_of = [](uint32_t dk) -> unsigned long long {      // the score units behind a key
        if (dk == 0xFFFFFFFFu) return 0ull;
        const uint32_t asc = ~dk;
        const uint32_t bits = (asc & 0x80000000u) ? (asc & 0x7FFFFFFFu) : ~asc;
        return (unsigned long long)score_units(__uint_as_float(bits));
    };
    // Score units of the entries with key <= cand (or < cand), summed over the warp.
    auto mass_upto = [&](uint32_t cand, bool strict) -> unsigned long long {
        unsigned long long ms = 0;
#pragma unroll
        for (int u = 0; u < KPL; ++u) {
            uint32_t h = hk[u];
            if (KPL > 32) asm volatile("" : "+r"(h));    // worked out again at every use: 64 more registers would not fit
            if (strict ? h < cand : h <= cand) ms += units_of(h);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ms += __shfl_xor_sync(0xFFFFFFFFu, ms, o);
        return ms;
    };
    // Smallest score key T such that the entries with key <= T are at least `target` many (by_count) or hold at
    // least `target` units of score: built bit by bit from the top, over the bits in which the keys differ.
    // Entries past the end carry the top key and no score: they are counted only where every real entry is.
    auto search = [&](unsigned long long target, bool by_count) -> uint32_t {
        uint32_t ans = k_and, todo = diff;
#pragma unroll 1
        while (todo) {
            const int bit = 31 - __clz((int)todo);
            todo &= ~(1u << bit);
            const uint32_t cand = (ans & ~(1u << bit)) | ((1u << bit) - 1u);
            unsigned long long have;
            if (!MASS || by_count) {
                int cnt = 0;
#pragma unroll
                for (int u = 0; u < KPL; ++u) cnt += hk[u] <= cand;
                have = (unsigned long long)warp_sum(cnt);
            } else {
                have = mass_upto(cand, false);
            }
            if (have >= target) ans &= ~(1u << bit); else ans |= 1u << bit;
        }
        return ans;
    };
    auto count_below = [&](uint32_t T) -> int {          // entries with a strictly better score than T
        int c = 0;
#pragma unroll
        for (int u = 0; u < KPL; ++u) c += hk[u] < T;
        return warp_sum(c);
    };

    // ---- how many entries reach the threshold, how many the budget allows --------------------------------------
    int k_beta = m;
    uint32_t T = ~0u;                                    // survivors: score key < T, and the first `need` entries of key T
    int need = 0;
    bool have_T = false;
    if (MASS && m > 0) {
        const unsigned long long total = mass_upto(~0u, false);
        const unsigned long long thr = ceil_muldiv(beta_ppm, total, 1000000ull);
        if (thr == 0) k_beta = 1;
        else {
            T = search(thr, false);
            const int c = count_below(T);
            const unsigned long long below = mass_upto(T, true);
            const unsigned long long each = units_of(T);                 // > 0: the entries of key T are needed
            need = (int)((thr - below + each - 1ull) / each);
            k_beta = c + need;
            have_T = true;
        }
    }
    int kc = k_beta;
    if (budget > 0) kc = min(kc, budget - (ln - m));
    kc = min(max(kc, 0), m);
    if (kc < m && kc > 0 && !(have_T && kc == k_beta)) {
        T = search((unsigned long long)kc, true);
        need = kc - count_below(T);
    }

    // ---- the survivor map, in index order: 32 entries a round, places by ballot ---------------------------------
    float* an = acc_new + (int64_t)m_idx * cap;
    int32_t* pn = pos_new + (int64_t)m_idx * cap;
    const uint32_t lt_mask = (1u << lane) - 1u;
    int first_drop = m;
    if (kc < m) {
        int base = 0, eq_base = 0;
#pragma unroll 2
        for (int j0 = 0; j0 < m; j0 += 32) {
            const int j = j0 + lane;
            const bool valid = j < m;
            const float sv = valid ? acc[lo + j] : 0.f;
            bool nf = false;
            const uint32_t h = valid ? desc_key(sv, &nf) : ~0u;
            const bool is_eq = valid && h == T;
            const uint32_t beq = __ballot_sync(0xFFFFFFFFu, is_eq);
            const bool kept = valid && kc > 0 && (h < T || (is_eq && eq_base + __popc(beq & lt_mask) < need));
            const uint32_t bk = __ballot_sync(0xFFFFFFFFu, kept);
            if (kept) {
                const int o = lo + base + __popc(bk & lt_mask);
                src[o] = lo + j;
                an[o] = sv;
                if (ps) pn[o] = (int32_t)my_pos[j];
            }
            const uint32_t bd = __ballot_sync(0xFFFFFFFFu, valid && !kept);
            if (first_drop == m && bd) first_drop = j0 + __ffs((int)bd) - 1;
            base += __popc(bk);
            eq_base += __popc(beq);
        }
    }
    const int new_len = lo + kc + (ln - hi);
    // rows that do not move (everything when nothing is evicted) and the rows behind the evictable range
    for (int o = lane; o < new_len; o += 32) {
        if (o < lo || kc >= m) {
            src[o] = o;
            if (o >= lo) { an[o] = acc[o]; if (ps) pn[o] = ps[o]; }
        } else if (o >= lo + kc) {
            const int sidx = hi + (o - lo - kc);
            src[o] = sidx;
            an[o] = acc[sidx];
            if (ps) pn[o] = ps[sidx];
        }
    }
    if (lane == 0) {
        meta[m_idx] = kc < m ? lo + first_drop : new_len;
        nout[m_idx] = new_len;
        len[m_idx] = new_len;
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
    float* acc_new = reinterpret_cast<float*>(wsb + L.off_acc);
    int32_t* pos_new = reinterpret_cast<int32_t*>(wsb + L.off_pos);

    const unsigned long long beta_ppm = (unsigned long long)llrint((double)beta * 1.0e6);
    const int heads = d->B * d->Hkv;
    lvlm_status st;
#define LVLM_PLAN_WARP_(KPL_, SMALL_, MASS_)                                                                     \
    (cudaFuncSetAttribute(kv_plan_warp_kernel<KPL_, MASS_>, cudaFuncAttributeMaxDynamicSharedMemorySize,              \
                          4 * 2 * KPL_ * 32 * 4) != cudaSuccess                                                       \
         ? LVLM_ERR_CUDA                                                                                             \
         : launch_kernel(kv_plan_warp_kernel<KPL_, MASS_>, dim3((heads + 3) / 4), dim3(128), 4 * 2 * KPL_ * 32 * 4,   \
                         stream, 1, acc_score, pos, len, e_lo, e_hi, heads, d->Hkv, d->cap, d->recent, SMALL_,        \
                         beta_ppm, budget, src_map, meta, nout, acc_new, pos_new, dev_status))
#define LVLM_PLAN_WARP(KPL_, SMALL_) \
    st = beta_ppm < 1000000ull ? LVLM_PLAN_WARP_(KPL_, SMALL_, true) : LVLM_PLAN_WARP_(KPL_, SMALL_, false)
    // With enough heads to fill the GPU with one warp each, a warp per head (no barrier in the searches); a CTA per
    // head otherwise, and for the heads whose entries do not fit a warp's registers.
    const bool many = heads >= 4 * 148;
    const int kpt = d->cap <= 4096 ? 4 : 16;
    int threads = ((d->cap + kpt - 1) / kpt + 31) / 32 * 32;
    threads = threads < 64 ? 64 : threads;
    int min_m = 0;                                       // heads the CTA kernel leaves to the warp kernel
    bool cta_kernel = true;
    if (many) {
        if (d->cap <= 512) LVLM_PLAN_WARP(16, 0);
        else if (d->cap <= 1024) LVLM_PLAN_WARP(32, 0);
        else if (d->cap <= 1536) LVLM_PLAN_WARP(48, 0);
        else if (d->cap <= 2048) LVLM_PLAN_WARP(64, 0);
        else LVLM_PLAN_WARP(32, 1);                      // long caches: the heads with up to 1024 evictable entries
        if (st != LVLM_OK) return st;
        cta_kernel = d->cap > 2048;                      // ... the others get a CTA each
        min_m = 32 * 32 + 1;
    }
    if (cta_kernel) {
        // a CTA per head, a thread holds 4 entries (caches up to 4096 rows) or 16; warps without entries leave at once
        st = kpt == 4 ? launch_kernel(kv_plan_kernel<4>, dim3(d->Hkv, d->B), dim3(threads), 0, stream, 1, acc_score, pos,
                                      len, e_lo, e_hi, d->Hkv, d->cap, d->recent, min_m, beta_ppm, budget, src_map,
                                      meta, nout, acc_new, pos_new, dev_status)
                      : launch_kernel(kv_plan_kernel<16>, dim3(d->Hkv, d->B), dim3(threads), 0, stream, 1, acc_score, pos,
                                      len, e_lo, e_hi, d->Hkv, d->cap, d->recent, min_m, beta_ppm, budget, src_map,
                                      meta, nout, acc_new, pos_new, dev_status);
    }
#undef LVLM_PLAN_WARP
#undef LVLM_PLAN_WARP_
    if (st != LVLM_OK) return st;
    CompactJob j;
    j.base0 = Kc; j.base1 = Vc; j.stride_b = kv_sb * 2; j.stride_g = kv_sh * 2; j.B = d->B; j.G = d->Hkv;
    j.V = kHeadDim / 8; j.src_map = src_map; j.maps_per_g = d->Hkv; j.map_stride = d->cap;
    j.meta = meta; j.meta_stride = 1; j.nout = nout; j.N = d->cap;
    j.side_dst[0] = acc_score; j.side_src[0] = acc_new;
    if (pos) { j.side_dst[1] = pos; j.side_src[1] = pos_new; }
    return launch_inplace_compact(j, stream);
}
