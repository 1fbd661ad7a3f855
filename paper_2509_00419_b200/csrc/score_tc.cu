// Tensor-core scoring kernels (tcgen05 + TMEM + TMA) for lvlm_score_tokens.
//
// The score of an image key is a column sum of softmax probabilities (Section 3.2.1,
// paragraph 3), so two passes over Q K^T are needed when the caller has no row normalisers:
//   pass 1 (MODE 0)  S = Q_tile K_tile^T with QUERIES on the TMEM lanes: every epilogue thread owns
//                    one query row and keeps its running max / sum over the key tiles -> lse.
//   pass 2 (MODE 1)  S^T = K_tile Q_tile^T with KEYS on the TMEM lanes: every epilogue thread owns
//                    one image key and adds exp2(logit - lse[row]) over all query rows and over
//                    the query heads of the KV group -> group-summed column sums.
// Both orientations are plain K-major operands (D is contiguous in Q and in K), so the same
// pipeline serves both: the A tile is loaded once, B tiles stream through a ring of shared-memory
// stages filled by TMA, one thread issues the MMAs into a double-buffered TMEM accumulator, and four
// epilogue warps drain it while the next tile is being multiplied.
#include "common.cuh"
#include "score.cuh"
#include "sm100.cuh"

namespace lvlm {

using namespace sm100;

constexpr int kTile = 128;                 // rows of A, rows of B, and K (= head dim)
constexpr int kStages = 2;                 // B-tile ring (two CTAs fit on an SM)
constexpr int kHalfBytes = kTile * 64 * 2; // one TMA box: 128 rows x 64 bf16 = 16 KB
constexpr int kTileBytes = 2 * kHalfBytes; // 32 KB
constexpr int kTcThreads = 320;            // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int kEpiThreads = 256;           // two warps per quarter of the TMEM lanes, 64 columns each
constexpr uint32_t kTmemCols = 256;        // two 128-column fp32 accumulators
constexpr float kLog2eT = 1.4426950408889634f;

struct ScoreTcArgs {
    int B, H, G, N, Nq, i0, n, q_lo, causal;
    float scale_log2;
    const float* lse_user;     // natural-log row normalisers from the caller, or NULL
    float* lse_ws;             // [B][H][Nq] log2-domain normalisers (pass 1 writes, pass 2 reads)
    float* partial;            // [B][Hkv * hsplit][n] column sums of each CTA row (pass 2 writes)
    int ksplit;                // pass 1: CTAs (one cluster) that share the key tiles of a query tile
    int nkt;                   // key tiles of pass 2 (its grid.x)
    int hsplit;                // CTAs that share the query heads of one KV group in pass 2
    int32_t* cnt;              // [B][key tiles] CTAs of pass 2 that have parked their sums (zero at its start)
    float* score;              // [B][n] head mean (written by the last CTA of a key tile)
    float* score_head;         // optional [B][Hkv] rows of n, head_stride apart
    int64_t head_stride;
    int32_t* dev_status;
};

struct TcSmem {
    uint64_t a_full, full[kStages], empty[kStages], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort;
    volatile int last;
    alignas(16) float lse_s[8][2][kTile / 2];  // per epilogue warp, per accumulator buffer: normalisers of its 64 columns
    float xm[kTile], xl[kTile];    // what the warps of the upper column half hand to the lower half
};

__device__ __forceinline__ void cluster_barrier_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(const float* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// 2^x on the special-function unit, one instruction (2 ulp, flush to zero: the scores tolerate 1e-3).
__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Pass 1, one chunk of 32 raw logits of a query row: columns [0, lim) are visible.  Updates the running
// (max, sum of 2^(logit*scale - max)).  Four partial sums keep the adds off one dependency chain.
__device__ __forceinline__ void rowstat_chunk(float* v, int lim, float scale_log2, float& m_run, float& l_run) {
    if (lim >= 32 && scale_log2 > 0.f) {
        // every column visible: the maximum is taken on the raw logits (a positive scale keeps the order)
        // and the scale is folded into the exponent's multiply-add
        float cmax = v[0];
#pragma unroll
        for (int c = 1; c < 32; ++c) cmax = fmaxf(cmax, v[c]);
        const float m_new = fmaxf(m_run, cmax * scale_log2);
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
            s0 += ex2_fast(fmaf(v[c], scale_log2, -m_new)); s1 += ex2_fast(fmaf(v[c + 1], scale_log2, -m_new));
            s2 += ex2_fast(fmaf(v[c + 2], scale_log2, -m_new)); s3 += ex2_fast(fmaf(v[c + 3], scale_log2, -m_new));
        }
        l_run = l_run * ex2_fast(m_run - m_new) + ((s0 + s1) + (s2 + s3));
        m_run = m_new;
        return;
    }
    float cmax = -INFINITY;
#pragma unroll
    for (int c = 0; c < 32; ++c) { v[c] = c < lim ? v[c] * scale_log2 : -INFINITY; cmax = fmaxf(cmax, v[c]); }
    const float m_new = fmaxf(m_run, cmax);
    if (m_new > -INFINITY) {
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
            s0 += ex2_fast(v[c] - m_new); s1 += ex2_fast(v[c + 1] - m_new);
            s2 += ex2_fast(v[c + 2] - m_new); s3 += ex2_fast(v[c + 3] - m_new);
        }
        l_run = l_run * ex2_fast(m_run - m_new) + ((s0 + s1) + (s2 + s3));
        m_run = m_new;
    }
}

// Pass 2, one chunk of 32 raw logits of a key against 32 query rows with normalisers ls (log2 domain):
// sum of the probabilities of the rows c >= first.
__device__ __forceinline__ float colsum_chunk(const float* v, const float* ls, int first, float scale_log2) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    if (first <= 0) {
        const float4* ls4 = reinterpret_cast<const float4*>(ls);         // 16-byte aligned: four normalisers a load
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
            const float4 l = ls4[c >> 2];
            s0 += ex2_fast(fmaf(v[c], scale_log2, -l.x)); s1 += ex2_fast(fmaf(v[c + 1], scale_log2, -l.y));
            s2 += ex2_fast(fmaf(v[c + 2], scale_log2, -l.z)); s3 += ex2_fast(fmaf(v[c + 3], scale_log2, -l.w));
        }
    } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            const float p = ex2_fast(fmaf(v[c], scale_log2, -ls[c]));
            s0 += c >= first ? p : 0.f;
        }
    }
    return (s0 + s1) + (s2 + s3);
}

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, TcSmem* sm, int32_t* dev_status) {
    if (sm->abort) return false;
    if (mbar_wait(bar, parity)) return true;
    sm->abort = 1;
    if (dev_status) atomicOr(dev_status, LVLM_DEV_TIMEOUT);
    return false;
}

template <int MODE>
__global__ void __launch_bounds__(kTcThreads, 2)
score_tc_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                const ScoreTcArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* sA = base;
    unsigned char* sB = base + kTileBytes;
    TcSmem* sm = reinterpret_cast<TcSmem*>(base + kTileBytes * (1 + kStages));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.z;
    const int nqt = (a.Nq + kTile - 1) / kTile;

    // ---- which tiles this CTA multiplies ---------------------------------------------------------
    int nt, h = 0, g = 0, qt = 0, kt = 0, qt_min = 0, nqt_vis = 0;
    const int h_first = MODE == 1 ? (blockIdx.y / a.hsplit) * a.G + (blockIdx.y % a.hsplit) * (a.G / a.hsplit) : 0;
    int t_off = 0;                                        // pass 1: first key tile of this CTA
    if (MODE == 0) {
        qt = blockIdx.x / a.ksplit; h = blockIdx.y; g = h / a.G;
        const int last_pos = a.q_lo + min(a.Nq, (qt + 1) * kTile) - 1;
        const int key_end = a.causal ? min(a.N, last_pos + 1) : a.N;
        const int nt_all = (key_end + kTile - 1) / kTile;
        const int per = (nt_all + a.ksplit - 1) / a.ksplit;
        t_off = min(nt_all, (int)(blockIdx.x % a.ksplit) * per);
        nt = min(nt_all, t_off + per) - t_off;
    } else {
        kt = blockIdx.x; g = blockIdx.y / a.hsplit;
        const int j0 = a.i0 + kt * kTile;
        qt_min = a.causal ? max(0, (j0 - a.q_lo) / kTile) : 0;
        nqt_vis = max(0, nqt - qt_min);
        nt = (a.G / a.hsplit) * nqt_vis;
    }

    if (threadIdx.x == 0) {
        mbar_init(&sm->a_full, 1);
        for (int s = 0; s < kStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sm->tmem_full[s], 1); mbar_init(&sm->tmem_empty[s], kEpiThreads); }
        sm->abort = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&qmap);
        prefetch_tmap(&kmap);
    }
    if (warp == 1) tmem_alloc(&sm->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    pdl_enter();                               // barriers and tensor memory are set up; now the inputs
    if (MODE == 0 && blockIdx.x == 0 && blockIdx.y == 0)      // pass 2 counts its CTAs per key tile from zero
        for (int i = threadIdx.x; i < a.nkt; i += blockDim.x) a.cnt[b * a.nkt + i] = 0;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0 && nt > 0) {
            mbar_arrive_expect_tx(&sm->a_full, kTileBytes);
            if (MODE == 0) {
                tma_load_4d(sA, &qmap, &sm->a_full, 0, h, qt * kTile, b);
                tma_load_4d(sA + kHalfBytes, &qmap, &sm->a_full, 64, h, qt * kTile, b);
            } else {
                tma_load_4d(sA, &kmap, &sm->a_full, 0, a.i0 + kt * kTile, g, b);
                tma_load_4d(sA + kHalfBytes, &kmap, &sm->a_full, 64, a.i0 + kt * kTile, g, b);
            }
            for (int t = 0; t < nt; ++t) {
                const int st = t % kStages;
                if (t >= kStages && !wait_or_abort(&sm->empty[st], ((t / kStages) - 1) & 1, sm, a.dev_status)) break;
                unsigned char* dst = sB + st * kTileBytes;
                mbar_arrive_expect_tx(&sm->full[st], kTileBytes);
                if (MODE == 0) {
                    tma_load_4d(dst, &kmap, &sm->full[st], 0, (t_off + t) * kTile, g, b);
                    tma_load_4d(dst + kHalfBytes, &kmap, &sm->full[st], 64, (t_off + t) * kTile, g, b);
                } else {
                    const int hh = h_first + t / nqt_vis, q2 = qt_min + t % nqt_vis;
                    tma_load_4d(dst, &qmap, &sm->full[st], 0, hh, q2 * kTile, b);
                    tma_load_4d(dst + kHalfBytes, &qmap, &sm->full[st], 64, hh, q2 * kTile, b);
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // all lanes run the loop (uniform operands), one elected lane issues
        if (nt > 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(kTile, kTile);
            const uint32_t a_addr = smem_u32(sA);
            uint64_t ad[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) ad[k] = smem_desc_sw128(a_addr + (k >> 2) * kHalfBytes + (k & 3) * 32);
            bool ok = __all_sync(0xFFFFFFFFu, wait_or_abort(&sm->a_full, 0, sm, a.dev_status));
            for (int t = 0; ok && t < nt; ++t) {
                const int st = t % kStages, buf = t & 1;
                const uint32_t b_addr = smem_u32(sB + st * kTileBytes);
                const uint32_t d_tmem = tmem_base + buf * kTile;
                uint64_t bd[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) bd[k] = smem_desc_sw128(b_addr + (k >> 2) * kHalfBytes + (k & 3) * 32);
                ok = wait_or_abort(&sm->full[st], (t / kStages) & 1, sm, a.dev_status);
                if (ok && t >= 2) ok = wait_or_abort(&sm->tmem_empty[buf], ((t / 2) - 1) & 1, sm, a.dev_status);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    mma_bf16_ss(d_tmem, ad[0], bd[0], idesc, 0u);
#pragma unroll
                    for (int k = 1; k < 8; ++k) mma_bf16_ss(d_tmem, ad[k], bd[k], idesc, 1u);
                    mma_commit(&sm->empty[st]);        // the stage may be refilled once these MMAs are done
                    mma_commit(&sm->tmem_full[buf]);   // ... and the accumulator may be drained
                }
                __syncwarp();
            }
        }
    } else {
        // ===== epilogue: warps 2..9; a warp reads TMEM lanes 32*(warp%4) .. +31, columns 64*half .. +63 =====
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;                 // TMEM lane = row of the A tile
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        float m_run = -INFINITY, l_run = 0.f, colsum = 0.f;
        const int my_pos = a.q_lo + qt * kTile + row;        // MODE 0: sequence position of my query
        const int my_key = a.i0 + kt * kTile + row;          // MODE 1: my key
        // row normalisers of a tile (MODE 1): every warp keeps its own copy of the tile's 128 values;
        // they are fetched one tile ahead so that the loads never sit on the critical path
        float lse_next[2] = {INFINITY, INFINITY};
        auto fetch_lse = [&](int t) {
            const int hh = h_first + t / nqt_vis, q2l = qt_min + t % nqt_vis;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int i = q2l * kTile + half * 64 + u * 32 + lane;
                float v = INFINITY;                            // rows past the window add nothing
                if (i < a.Nq) {
                    const int64_t idx = ((int64_t)b * a.H + hh) * a.Nq + i;
                    v = a.lse_user ? a.lse_user[idx] * kLog2eT : __ldcg(a.lse_ws + idx);
                }
                lse_next[u] = v;
            }
        };
        if (MODE == 1 && nt > 0) fetch_lse(0);
        for (int t = 0; t < nt; ++t) {
            const int buf = t & 1;
            int q2 = 0;
            if (MODE == 1) {
                q2 = qt_min + t % nqt_vis;
#pragma unroll
                for (int u = 0; u < 2; ++u) sm->lse_s[warp - 2][buf][u * 32 + lane] = lse_next[u];
                if (t + 1 < nt) fetch_lse(t + 1);
                __syncwarp();
            }
            if (!wait_or_abort(&sm->tmem_full[buf], (t / 2) & 1, sm, a.dev_status)) break;
            tc_fence_after();
#pragma unroll 1
            for (int c2 = 0; c2 < 2; ++c2) {
                const int c4 = half * 2 + c2;                  // 32-column chunk of the tile
                // nothing to do where the tile sticks out of the window: a warp whose 32 query rows lie past
                // it (pass 1), a chunk whose 32 query rows lie past it (pass 2)
                if (MODE == 0 && qt * kTile + quarter * 32 >= a.Nq) continue;
                if (MODE == 1 && q2 * kTile + c4 * 32 >= a.Nq) continue;
                float v[32];
                tmem_ld32(lane_addr + buf * kTile + c4 * 32, v);
                tmem_ld_wait();
                if (MODE == 0) {
                    const int jb = (t_off + t) * kTile + c4 * 32;
                    const int lim = min(a.N, a.causal ? my_pos + 1 : a.N) - jb;    // columns < lim are visible
                    rowstat_chunk(v, lim, a.scale_log2, m_run, l_run);
                } else {
                    const int ib = q2 * kTile + c4 * 32;                           // first query row of the chunk
                    // query i sees my key iff my_key <= q_lo + i  <=>  c >= my_key - q_lo - ib
                    const int first = a.causal ? my_key - a.q_lo - ib : 0;
                    colsum += colsum_chunk(v, &sm->lse_s[warp - 2][buf][c2 * 32], first, a.scale_log2);
                }
            }
            tc_fence_before();
            mbar_arrive(&sm->tmem_empty[buf]);
        }
        // the two column halves of a row meet in shared memory; every epilogue thread takes this path,
        // also after a timeout, so that the barriers and the counters always see all of them
        if (half == 1) { sm->xm[row] = MODE == 0 ? m_run : colsum; sm->xl[row] = l_run; }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (MODE == 0) {
            if (half == 0) {
                const float m1 = sm->xm[row], l1 = sm->xl[row];
                const float M = fmaxf(m_run, m1);
                float L = 0.f;
                if (m_run > -INFINITY) L += l_run * exp2f(m_run - M);
                if (m1 > -INFINITY) L += l1 * exp2f(m1 - M);
                const int i = qt * kTile + row;
                if (a.ksplit == 1) {
                    if (!sm->abort && i < a.Nq) a.lse_ws[((int64_t)b * a.H + h) * a.Nq + i] = M + log2f(L);
                } else {                                   // the cluster combines below
                    sm->xm[row] = M; sm->xl[row] = L;
                }
            }
        } else {
            if (half == 0) colsum += sm->xm[row];
            const int Hkv = a.H / a.G, P = Hkv * a.hsplit;       // CTA rows per sequence
            const int jl = kt * kTile + row;
            if (half == 0 && jl < a.n) a.partial[((int64_t)b * P + blockIdx.y) * a.n + jl] = colsum;
            // the last CTA of this key tile adds the rows in row order: head mean and group sums
            __threadfence();
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (threadIdx.x == 64) sm->last = atomicAdd(&a.cnt[b * gridDim.x + kt], 1) == P - 1;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (sm->last && half == 0) {
                __threadfence();
                if (jl < a.n) {
                    float tot = 0.f;
                    for (int gg = 0; gg < Hkv; ++gg) {
                        float gs = 0.f;
                        for (int pp = 0; pp < a.hsplit; ++pp)
                            gs += __ldcg(a.partial + ((int64_t)b * P + gg * a.hsplit + pp) * a.n + jl);
                        if (a.score_head) a.score_head[((int64_t)b * Hkv + gg) * a.head_stride + jl] = gs;
                        tot += gs;
                    }
                    const float sc = tot * (1.0f / (float)a.H);
                    a.score[(int64_t)b * a.n + jl] = sc;
                    if (a.dev_status && (__float_as_uint(sc) & 0x7F800000u) == 0x7F800000u)
                        atomicOr(a.dev_status, LVLM_DEV_NONFINITE);
                }
                if (threadIdx.x == 64) a.cnt[b * gridDim.x + kt] = 0;
            }
        }
    }
    // ---- common exit: everyone meets, then the allocating warp frees the tensor memory ----------
    tc_fence_before();
    __syncthreads();
    if (MODE == 0 && a.ksplit > 1) {
        // the CTAs of the cluster hold (max, sum) of their share of the keys for the same 128 rows:
        // rank 0 adds them in rank order and writes the normalisers
        cluster_barrier_all();
        if (blockIdx.x % a.ksplit == 0 && threadIdx.x >= 64 && threadIdx.x < 64 + kTile) {
            const int row = threadIdx.x - 64;
            float M = -INFINITY;
            for (int r = 0; r < a.ksplit; ++r) M = fmaxf(M, ld_cluster_f32(&sm->xm[row], r));
            float L = 0.f;
            for (int r = 0; r < a.ksplit; ++r) {
                const float m = ld_cluster_f32(&sm->xm[row], r);
                if (m > -INFINITY) L += ld_cluster_f32(&sm->xl[row], r) * exp2f(m - M);
            }
            const int i = (blockIdx.x / a.ksplit) * kTile + row;
            if (!sm->abort && i < a.Nq) a.lse_ws[((int64_t)b * a.H + blockIdx.y) * a.Nq + i] = M + log2f(L);
        }
        cluster_barrier_all();
    }
    if (sm->abort) {                              // let copies still in flight land before leaving
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

lvlm_status launch_score_tc(const void* Q, const void* K, const float* lse, const lvlm_dims* d,
                            const ScoreStrides& st, float scale, float* lse_ws, float* partial,
                            int32_t* cnt, float* score, float* score_head, int32_t* dev_status,
                            cudaStream_t stream, bool normalisers_ready) {
    const int Nq = d->q_hi - d->q_lo;
    CUtensorMap qmap, kmap;
    {
        const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)d->H, (uint64_t)Nq, (uint64_t)d->B};
        const uint64_t strides[3] = {(uint64_t)st.q_sh * 2, (uint64_t)st.q_sn * 2, (uint64_t)st.q_sb * 2};
        const uint32_t box[4] = {64, 1, (uint32_t)kTile, 1};
        if (!make_tmap_bf16(&qmap, Q, 4, dims, strides, box)) return LVLM_ERR_CUDA;
    }
    {
        const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)d->N, (uint64_t)d->Hkv, (uint64_t)d->B};
        const uint64_t strides[3] = {(uint64_t)kHeadDim * 2, (uint64_t)st.kv_sh * 2, (uint64_t)st.kv_sb * 2};
        const uint32_t box[4] = {64, (uint32_t)kTile, 1, 1};
        if (!make_tmap_bf16(&kmap, K, 4, dims, strides, box)) return LVLM_ERR_CUDA;
    }
    ScoreTcArgs a;
    a.B = d->B; a.H = d->H; a.G = d->H / d->Hkv; a.N = d->N; a.Nq = Nq; a.i0 = d->i0; a.n = d->n;
    a.q_lo = d->q_lo; a.causal = d->causal; a.scale_log2 = scale * kLog2eT;
    a.lse_user = lse; a.lse_ws = lse_ws; a.partial = partial; a.dev_status = dev_status;
    a.cnt = cnt; a.score = score; a.score_head = score_head;
    a.head_stride = d->head_stride ? d->head_stride : (int64_t)d->n;
    const size_t smem = 1024 + (size_t)kTileBytes * (1 + kStages) + sizeof(TcSmem);
    const int nqt = (Nq + kTile - 1) / kTile, nkt = (d->n + kTile - 1) / kTile;
    // pass 2: the query heads of a KV group can be shared out over hs CTAs (hs divides G).  More CTAs
    // fill the GPU, fewer amortise a CTA's fixed cost over more tiles: take the hs with the smallest
    // estimate waves x (fixed + tiles per CTA x per-tile), 296 CTAs to a wave (two per SM).
    int hsplit = 1;
    {
        double best = 1e30;
        for (int hs = 1; hs <= a.G; ++hs) {
            if (a.G % hs) continue;
            const int64_t ctas = (int64_t)nkt * d->Hkv * d->B * hs;
            const double waves = (double)((ctas + 295) / 296);
            const double est = waves * (5.0 + 0.6 * (a.G / hs) * nqt);
            if (est < best - 1e-9) { best = est; hsplit = hs; }
        }
    }
    a.hsplit = hsplit; a.nkt = nkt; a.ksplit = 1;
    const bool skip_pass1 = lse != nullptr || normalisers_ready;
    if (skip_pass1) LVLM_RETURN_IF_CUDA(cudaMemsetAsync(cnt, 0, (size_t)d->B * nkt * 4, stream));
    if (!skip_pass1) {
        LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(score_tc_kernel<0>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        // pass 1: when query tiles x heads do not fill the GPU, a cluster of CTAs shares the key tiles
        // (the split with the smallest estimate waves x (fixed + key tiles per CTA x per-tile), as for pass 2)
        int ksplit = 1;
        const int max_kt = (d->N + kTile - 1) / kTile;
        {
            double best = 1e30;
            for (int ks = 1; ks <= 8 && ks <= max_kt; ++ks) {
                const int64_t ctas = (int64_t)nqt * d->H * d->B * ks;
                const double waves = (double)((ctas + 295) / 296);
                const double est = waves * (5.0 + 0.6 * ((max_kt + ks - 1) / ks));
                if (est < best - 1e-9) { best = est; ksplit = ks; }
            }
        }
        a.ksplit = ksplit;
        const lvlm_status s0 = launch_kernel(score_tc_kernel<0>, dim3(nqt * ksplit, d->H, d->B), dim3(kTcThreads),
                                             smem, stream, ksplit, qmap, kmap, a);
        if (s0 != LVLM_OK) return s0;
    }
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(score_tc_kernel<1>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    return launch_kernel(score_tc_kernel<1>, dim3(nkt, d->Hkv * hsplit, d->B), dim3(kTcThreads), smem, stream, 1,
                         qmap, kmap, a);
}

}  // namespace lvlm
