// lvlm_decode_attn: one generated token attends to every cached key and value of its KV head
// (Section 3.2.2, paragraph 1), over caches whose lengths differ per (sequence, KV head) after
// compression.  HBM-bound: every K and V row is read once and shared by the G query heads of
// the group.
//
// One launch, split-K inside thread-block clusters.  The S CTAs of a cluster share one (sequence,
// KV head): its key tiles are cut into S equal runs, so a ragged cache costs what its own length
// costs.  A CTA is one producer warp and four compute warps around a ring of shared-memory stages
// of 64 keys: the producer fetches the K and V rows of a stage with four TMA tile copies (128-byte
// swizzle, so that ldmatrix is conflict free; completion counted by an mbarrier), a compute warp
// takes 16 keys of the stage, multiplies them with small tensor-core MMAs (the G query heads of the
// group are the rows of a 16-row tile) and keeps an online softmax per head, so the main loop has no
// block barrier.  With d->cache_stable the first lap of the ring is fetched before the kernel waits
// for the one ahead of it in the stream.  The warps of a CTA are merged in warp order
// in shared memory; the CTAs of the cluster then read each other's (max, sum, output) through
// distributed shared memory in rank order, each finishing a slice of the output channels and the
// acc_score entries of its own keys, whose scaled logits it has kept in shared memory (in the
// workspace when a run is too long for that).
#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace lvlm {

using namespace sm100;

constexpr int kDecWarps = 4;                         // compute warps
constexpr int kDecThreads = (kDecWarps + 1) * 32;    // ... and the producer warp
constexpr int kTileKeys = 16;                        // keys per warp tile
constexpr int kStageKeys = kDecWarps * kTileKeys;    // keys per stage
constexpr int kBoxBytes = kStageKeys * 128;          // one TMA box: 64 keys x 64 channels
constexpr int kStageBytes = 4 * kBoxBytes;           // K low half, K high half, V low half, V high half
constexpr int kStagesDec = 3;
constexpr int kRingBytes = kStagesDec * kStageBytes;
constexpr int kDecTargetCtas = 2 * 148;              // CTAs wanted in flight: two per SM of a 148-SM part
constexpr int kDecMaxCluster = 8;                    // portable cluster size
constexpr int kDecMinTiles = 2;                      // a CTA's run is not made shorter than this by splitting
constexpr int kDecLogitBytes = 12 * 1024;            // scaled logits of a CTA's own keys kept in shared memory
constexpr float kLog2e = 1.4426950408889634f;

struct DecodeLayout { int S; size_t off_s, total; };

static bool decode_layout(const lvlm_dims* d, DecodeLayout* L) {
    if (!d || d->B <= 0 || d->H <= 0 || d->Hkv <= 0 || d->H % d->Hkv || d->cap <= 0) return false;
    // cluster size: the power of two that brings the grid closest to the target without going
    // over it, as long as a full cache still gives every CTA a few tiles
    const int64_t heads = (int64_t)d->B * d->Hkv;
    const int tiles = (d->cap + kTileKeys - 1) / kTileKeys;
    int S = 1;
    while (S < kDecMaxCluster && heads * (2 * S) <= kDecTargetCtas && tiles / (2 * S) >= kDecMinTiles) S *= 2;
    L->S = S;
    size_t off = 0;
    L->off_s = off; off = align_up(off + (size_t)d->B * d->H * d->cap * 4, 256);
    L->total = off;
    return true;
}

size_t decode_attn_workspace(const lvlm_dims* d) {
    DecodeLayout L;
    return decode_layout(d, &L) ? L.total : 0;
}

// ---- thread-block cluster primitives ---------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Every thread of every CTA of the cluster arrives and waits; shared-memory writes made before it
// are visible to the other CTAs after it.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
// Address of my shared-memory location `saddr` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ float dsmem_ld(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D (16x8 fp32) += A (16x16 bf16, row) * B (16x8 bf16, col)
__device__ __forceinline__ void mma_16816(float* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct DecodeArgs {
    const __nv_bfloat16* q; __nv_bfloat16* Kc; __nv_bfloat16* Vc; int32_t* len;
    const __nv_bfloat16* k_new; const __nv_bfloat16* v_new; float* acc_score; __nv_bfloat16* out;
    int H, Hkv, cap, S;
    int early;               // the cache and len are not written by the kernel ahead: fetch before waiting for it
    int logit_keys;          // keys of a run whose logits fit in shared memory (0: they go to ws_s)
    int64_t kv_sb, kv_sh;
    float scale_log2;
    float* ws_s;             // [B*H][cap] scaled logits (log2 domain), only with acc_score and a long run
    int32_t* dev_status;
};

// Offset inside a stage of the 16-byte chunk `ch` (0..15) of key row `r` (0..63): K or V half boxes of 64
// channels, rows of 128 bytes, chunks XOR-swizzled with the row as the TMA copy wrote them.
__device__ __forceinline__ uint32_t stage_off(int r, int ch) {
    return (uint32_t)((ch >> 3) * kBoxBytes + r * 128 + (((ch & 7) ^ (r & 7)) << 4));
}

// grid.x = heads * S, clusters of S CTAs along x: cluster = (sequence, KV head), rank = run of tiles.
// CL = false: one CTA per head and no cluster instruction in the kernel at all.
template <int G, bool CL>
__global__ void __launch_bounds__(kDecThreads, 2)
decode_cluster_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap,
                      const DecodeArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* s_acc = reinterpret_cast<float*>(smem);                      // [slots][G][128]; slot 0 = this CTA's output (the ring, once it is done)
    float* s_wm = reinterpret_cast<float*>(smem + kRingBytes);          // [4 warps][8 heads] running max
    float* s_wl = s_wm + kDecWarps * 8;                                 // [4 warps][8 heads] running sum
    float* s_M = s_wl + kDecWarps * 8;                                  // [8] this CTA's max per head
    float* s_L = s_M + 8;                                               // [8] this CTA's sum per head
    float* s_FM = s_L + 8;                                              // [8] cluster-wide max
    float* s_FI = s_FM + 8;                                             // [8] 1 / cluster-wide sum
    float* s_rm = s_FI + 8;                                             // [S][8] max of every CTA of the cluster
    float* s_rl = s_rm + 8 * kDecMaxCluster;                            // [S][8] sum of every CTA
    uint64_t* s_full = reinterpret_cast<uint64_t*>(s_rl + 8 * kDecMaxCluster);   // [kStagesDec]
    uint64_t* s_empty = s_full + kStagesDec;                            // [kStagesDec]
    float* s_logit = reinterpret_cast<float*>(s_empty + kStagesDec + 1);          // [G][logit_keys]
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 32) { prefetch_tmap(&kmap); prefetch_tmap(&vmap); }     // the descriptors start their way first
    if (tid == 0) {
        for (int s = 0; s < kStagesDec; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], kDecWarps); }
        s_abort = 0;
        fence_barrier_init();
    }
    __syncthreads();
    // With a.early the first key/value stages and the length are fetched while the kernel ahead in the
    // stream is still finishing; q, k_new, v_new and every write come after the wait in any case.
    if (!a.early) pdl_enter();
    const int S = CL ? a.S : 1, H = a.H, cap = a.cap;
    const int hd = blockIdx.x / S;
    const int rank = CL ? (int)cluster_ctarank() : 0;
    const int b = hd / a.Hkv, g = hd % a.Hkv, h0 = g * G;

    // ---- this head's length; every CTA of the cluster takes the same decisions ---------------------------
    int ln = a.len[hd];
    const bool bad = ln < 0 || ln > cap;
    if (bad) ln = 0;
    const bool app = a.k_new != nullptr && !bad && ln < cap;
    if (rank == 0 && tid == 0 && a.dev_status && (bad || (a.k_new != nullptr && !bad && !app)))
        atomicOr(a.dev_status, LVLM_DEV_BOUNDS);                        // bad length, or append at capacity
    const int lne = ln + (app ? 1 : 0);
    if (lne == 0) {                                                     // no key at all: zeros
        if (a.early) pdl_enter();
        if (rank == 0)
            for (int i = tid; i < G * kHeadDim; i += kDecThreads)
                a.out[(int64_t)(b * H + h0) * kHeadDim + i] = __float2bfloat16_rn(0.f);
        return;
    }
    const int nt = (lne + kTileKeys - 1) / kTileKeys;
    int per = (nt + S - 1) / S;
    if (per >= kDecWarps) per = (per + kDecWarps - 1) / kDecWarps * kDecWarps;   // whole stages where the run is long enough
    const int t_lo = min(nt, rank * per), t_hi = min(nt, t_lo + per);   // my run of tiles
    const int nstage = (t_hi - t_lo + kDecWarps - 1) / kDecWarps;
    const uint32_t ring = smem_u32(smem);
    volatile int* abort_flag = &s_abort;
    auto wait_on = [&](uint64_t* bar, uint32_t parity) -> bool {
        if (*abort_flag) return false;
        if (mbar_wait(bar, parity)) return true;
        *abort_flag = 1;
        if (a.dev_status) atomicOr(a.dev_status, LVLM_DEV_TIMEOUT);
        return false;
    };

    float o[16][2];                            // head `row`, columns nt*8 + qd*2 + {0,1}
#pragma unroll
    for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;      // of head `row`; l_run is this lane's share of the sum
    const int row = lane >> 2, qd = lane & 3;

    if (warp == kDecWarps) {
        // ---- producer: four tile copies per stage ---------------------------------------------------------
        auto issue = [&](int s) {
            unsigned char* st = smem + (s % kStagesDec) * kStageBytes;
            const int j0 = (t_lo + s * kDecWarps) * kTileKeys;
            mbar_arrive_expect_tx(&s_full[s % kStagesDec], kStageBytes);
            tma_load_4d(st, &kmap, &s_full[s % kStagesDec], 0, j0, g, b);
            tma_load_4d(st + kBoxBytes, &kmap, &s_full[s % kStagesDec], 64, j0, g, b);
            tma_load_4d(st + 2 * kBoxBytes, &vmap, &s_full[s % kStagesDec], 0, j0, g, b);
            tma_load_4d(st + 3 * kBoxBytes, &vmap, &s_full[s % kStagesDec], 64, j0, g, b);
        };
        if (lane == 0) {
            for (int s = 0; s < kStagesDec && s < nstage; ++s) issue(s);
        }
        if (a.early) pdl_enter();
        if (lane == 0) {
            for (int s = kStagesDec; s < nstage; ++s) {
                if (!wait_on(&s_empty[s % kStagesDec], (uint32_t)(s / kStagesDec - 1) & 1u)) break;
                issue(s);
            }
        }
    } else {
        if (a.acc_score) {                     // my keys' acc_score entries: needed at the very end, fetched now
            const float* acc = a.acc_score + (int64_t)hd * cap;
            const int j_lo = t_lo * kTileKeys, j_hi = min(lne, t_hi * kTileKeys);
            for (int j = j_lo + tid * 32; j < j_hi; j += kDecWarps * 32 * 32) prefetch_l2(acc + j);
        }
        if (a.early) pdl_enter();
        const int64_t kv_off = (int64_t)b * a.kv_sb + (int64_t)g * a.kv_sh;
        __nv_bfloat16* Kseq = a.Kc + kv_off;
        __nv_bfloat16* Vseq = a.Vc + kv_off;
        const __nv_bfloat16* kn = app ? a.k_new + (int64_t)hd * kHeadDim : nullptr;
        const __nv_bfloat16* vn = app ? a.v_new + (int64_t)hd * kHeadDim : nullptr;
        // query fragments: heads of the group are rows 0..G-1 of a 16-row A tile
        uint32_t qa[8][2];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = qa[ks][1] = 0u;
            if (row < G) {
                const uint32_t* qp = reinterpret_cast<const uint32_t*>(a.q + (int64_t)(b * H + h0 + row) * kHeadDim);
                qa[ks][0] = __ldg(qp + ks * 8 + qd);
                qa[ks][1] = __ldg(qp + ks * 8 + 4 + qd);
            }
        }
        for (int s = 0; s < nstage; ++s) {
            const bool ok = wait_on(&s_full[s % kStagesDec], (uint32_t)(s / kStagesDec) & 1u);
            const int t = t_lo + s * kDecWarps + warp;
            if (ok && t < t_hi) {
                const uint32_t st = ring + (s % kStagesDec) * kStageBytes;      // K boxes; the V boxes follow
                const int r0 = warp * kTileKeys;                               // my rows of the stage
                const int j0 = t * kTileKeys;
                if (app && ln >= j0 && ln < j0 + kTileKeys) {
                    // the appended row: into its place of the tile and into the cache
                    const int rr = r0 + ln - j0, ch = lane & 15;
                    const uint4 x = *reinterpret_cast<const uint4*>((lane < 16 ? kn : vn) + ch * 8);
                    const uint32_t off = (lane < 16 ? 0 : 2 * kBoxBytes) + stage_off(rr, ch);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(st + off), "r"(x.x), "r"(x.y), "r"(x.z), "r"(x.w) : "memory");
                    *reinterpret_cast<uint4*>((lane < 16 ? Kseq : Vseq) + (int64_t)ln * kHeadDim + ch * 8) = x;
                }
                if (j0 + kTileKeys > lne) {
                    // V rows past the last key hold whatever the cache holds: zero them, their weight is zero
                    for (int e = lane; e < (j0 + kTileKeys - lne) * 16; e += 32) {
                        const int rr = r0 + (lne - j0) + (e >> 4), ch = e & 15;
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(st + 2 * kBoxBytes + stage_off(rr, ch)), "r"(0u) : "memory");
                    }
                }
                __syncwarp();
                // ---- S = Q K^T for 16 keys -------------------------------------------------------------------
                float sc[2][4];
#pragma unroll
                for (int i = 0; i < 2; ++i) sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
                {
                    const int mi = lane >> 3, r8 = lane & 7;
                    const int key = r0 + (mi >> 1) * 8 + r8;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const int chunkc = 2 * ks + (mi & 1);
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4(st + stage_off(key, chunkc), b0, b1, b2, b3);
                        mma_16816(sc[0], qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
                        mma_16816(sc[1], qa[ks][0], 0u, qa[ks][1], 0u, b2, b3);
                    }
                }
                // ---- online softmax of head `row` over the tile's keys -------------------------------------------
                float tmax = -INFINITY;
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc) {
                        const int j = j0 + i * 8 + qd * 2 + cc;
                        float v = sc[i][cc] * a.scale_log2;
                        if (j >= lne) v = -INFINITY;
                        sc[i][cc] = v;
                        tmax = fmaxf(tmax, v);
                        if (a.acc_score && row < G && j < lne) {
                            if (a.logit_keys) s_logit[row * a.logit_keys + (j - t_lo * kTileKeys)] = v;
                            else a.ws_s[(int64_t)(b * H + h0 + row) * cap + j] = v;
                        }
                    }
                tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, 1));
                tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, 2));
                const float m_new = fmaxf(m_run, tmax);          // finite: every tile has a valid key
                const float corr = exp2f(m_run - m_new);
                m_run = m_new;
                float p[2][2];
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc) p[i][cc] = exp2f(sc[i][cc] - m_new);
                l_run = l_run * corr + (p[0][0] + p[0][1]) + (p[1][0] + p[1][1]);
#pragma unroll
                for (int i = 0; i < 16; ++i) { o[i][0] *= corr; o[i][1] *= corr; }
                // ---- O += P V -----------------------------------------------------------------------------------
                // P is split into a bf16 head and a bf16 remainder so that the product keeps ~16 bits
                const uint32_t pa0 = pack_bf16(p[0][0], p[0][1]), pa2 = pack_bf16(p[1][0], p[1][1]);
                const uint32_t pr0 = pack_bf16(p[0][0] - bf16_lo(pa0), p[0][1] - bf16_hi(pa0));
                const uint32_t pr2 = pack_bf16(p[1][0] - bf16_lo(pa2), p[1][1] - bf16_hi(pa2));
                {
                    const int mi = lane >> 3, r8 = lane & 7;
                    const int key = r0 + (mi & 1) * 8 + r8;
#pragma unroll
                    for (int dp = 0; dp < 8; ++dp) {
                        const int chunkc = 2 * dp + (mi >> 1);
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4_trans(st + 2 * kBoxBytes + stage_off(key, chunkc), b0, b1, b2, b3);
                        // rows 8..15 of the MMA tile are padding: their accumulators are thrown away
                        float d0[4] = {o[2 * dp][0], o[2 * dp][1], 0.f, 0.f};
                        float d1[4] = {o[2 * dp + 1][0], o[2 * dp + 1][1], 0.f, 0.f};
                        mma_16816(d0, pa0, 0u, pa2, 0u, b0, b1);
                        mma_16816(d1, pa0, 0u, pa2, 0u, b2, b3);
                        mma_16816(d0, pr0, 0u, pr2, 0u, b0, b1);
                        mma_16816(d1, pr0, 0u, pr2, 0u, b2, b3);
                        o[2 * dp][0] = d0[0]; o[2 * dp][1] = d0[1];
                        o[2 * dp + 1][0] = d1[0]; o[2 * dp + 1][1] = d1[1];
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_empty[s % kStagesDec]);
        }
    }
    // every copy issued has landed: the compute warps have waited for each stage; the ring is free
    __syncthreads();
    if (s_abort) {                             // a wait gave up: copies may still be in flight, let them land
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }

    // ---- merge the four warps in warp order ------------------------------------------------------------
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
    if (warp < kDecWarps && row < G && qd == 0) { s_wm[warp * 8 + row] = m_run; s_wl[warp * 8 + row] = l_run; }
    __syncthreads();
    {
        // kSlots warps write side by side, the others add to them in warp order; the slots are added
        // in slot order when they are folded into slot 0
        constexpr int kSlots = G <= 4 ? 4 : 2;
        float Mh = -INFINITY;
        if (row < G) {
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) Mh = fmaxf(Mh, s_wm[w * 8 + row]);
        }
        const float f = (row < G && m_run > -INFINITY) ? exp2f(m_run - Mh) : 0.f;
#pragma unroll
        for (int rnd = 0; rnd < kDecWarps / kSlots; ++rnd) {
            if (warp / kSlots == rnd && row < G) {
                float* slot = s_acc + (warp % kSlots) * (G * kHeadDim);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float2* dst = reinterpret_cast<float2*>(slot + row * kHeadDim + i * 8 + qd * 2);
                    float2 v = make_float2(o[i][0] * f, o[i][1] * f);
                    if (rnd > 0) { const float2 old = *dst; v.x += old.x; v.y += old.y; }
                    *dst = v;
                }
            }
            __syncthreads();
        }
#pragma unroll
        for (int hh = 0; hh < G && tid < kHeadDim; ++hh) {  // thread = channel
            float v = s_acc[hh * kHeadDim + tid];
#pragma unroll
            for (int sl = 1; sl < kSlots; ++sl) v += s_acc[sl * (G * kHeadDim) + hh * kHeadDim + tid];
            s_acc[hh * kHeadDim + tid] = v;
        }
        if (tid < G) {
            float M2 = -INFINITY;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) M2 = fmaxf(M2, s_wm[w * 8 + tid]);
            float Ls = 0.f;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) {
                const float mw = s_wm[w * 8 + tid];
                if (mw > -INFINITY) Ls += s_wl[w * 8 + tid] * exp2f(mw - M2);
            }
            s_M[tid] = M2;
            s_L[tid] = Ls;
        }
    }

    // ---- combine the CTAs of the cluster in rank order through distributed shared memory ----------------
    if (CL) cluster_sync_all(); else __syncthreads();
    // my slice of the output channels: element (hh, d) with hh*128 + d = rank*128 + tid (+ S*128 ...).
    // A thread fetches what it needs from every CTA in one go (max, sum and its channel) and
    // works out the weights itself, so there is one round trip and no block barrier on this path.
    for (int idx = rank * kDecThreads + tid; idx < G * kHeadDim; idx += S * kDecThreads) {
        const int hh = idx >> 7;
        const uint32_t a_o = (uint32_t)__cvta_generic_to_shared(s_acc + idx);
        const uint32_t a_m = (uint32_t)__cvta_generic_to_shared(s_M + hh);
        const uint32_t a_l = (uint32_t)__cvta_generic_to_shared(s_L + hh);
        float x[kDecMaxCluster], m[kDecMaxCluster], l[kDecMaxCluster];
#pragma unroll
        for (int r = 0; r < kDecMaxCluster; ++r) {
            x[r] = 0.f; m[r] = -INFINITY; l[r] = 0.f;
            if (r < S) {
                if (CL) {
                    x[r] = dsmem_ld(dsmem_addr(a_o, r));
                    m[r] = dsmem_ld(dsmem_addr(a_m, r));
                    l[r] = dsmem_ld(dsmem_addr(a_l, r));
                } else {                       // a head with one CTA: its own shared memory, read directly
                    x[r] = s_acc[idx]; m[r] = s_M[hh]; l[r] = s_L[hh];
                }
            }
        }
        float FM = -INFINITY;
#pragma unroll
        for (int r = 0; r < kDecMaxCluster; ++r) FM = fmaxf(FM, m[r]);
        float v = 0.f, Ls = 0.f;
#pragma unroll
        for (int r = 0; r < kDecMaxCluster; ++r) {
            const float w = m[r] > -INFINITY ? exp2f(m[r] - FM) : 0.f;
            v += x[r] * w;
            Ls += l[r] * w;
        }
        a.out[(int64_t)(b * H + h0) * kHeadDim + idx] = __float2bfloat16_rn(Ls > 0.f ? v / Ls : 0.f);
    }
    if (CL && a.acc_score && tid < 8 * S) {    // (max, sum) of every CTA and head, for the acc_score update
        const int r = tid >> 3, hh = tid & 7;
        float m = -INFINITY, l = 0.f;
        if (hh < G) {
            m = dsmem_ld(dsmem_addr((uint32_t)__cvta_generic_to_shared(s_M + hh), r));
            l = dsmem_ld(dsmem_addr((uint32_t)__cvta_generic_to_shared(s_L + hh), r));
        }
        s_rm[tid] = m;
        s_rl[tid] = l;
    }
    if (CL) cluster_arrive();                  // my reads of the other CTAs' shared memory are done
    // the probabilities of my own keys go to acc_score
    if (a.acc_score) {
        if (!CL) {                             // one CTA: its own (max, sum) are the head's
            if (tid < G) { s_FM[tid] = s_M[tid]; s_FI[tid] = s_L[tid] > 0.f ? 1.0f / s_L[tid] : 0.f; }
        } else {
            __syncthreads();
        }
        if (CL && tid < G) {
            float FM = -INFINITY;
            for (int r = 0; r < S; ++r) FM = fmaxf(FM, s_rm[r * 8 + tid]);
            float Ls = 0.f;
            for (int r = 0; r < S; ++r) {
                const float m = s_rm[r * 8 + tid];
                if (m > -INFINITY) Ls += s_rl[r * 8 + tid] * exp2f(m - FM);
            }
            s_FM[tid] = FM;
            s_FI[tid] = Ls > 0.f ? 1.0f / Ls : 0.f;
        }
        __syncthreads();
        float* acc = a.acc_score + (int64_t)hd * cap;
        float il[G], mx[G];
#pragma unroll
        for (int hh = 0; hh < G; ++hh) { mx[hh] = s_FM[hh]; il[hh] = s_FI[hh]; }
        const int j_lo = t_lo * kTileKeys, j_hi = min(lne, t_hi * kTileKeys);
        // four keys per thread per round: 4 (G + 1) independent loads in flight
        for (int j0 = j_lo + tid; j0 < j_hi; j0 += 4 * kDecThreads) {
            float lg[4][G], old[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = j0 + u * kDecThreads;
                old[u] = 0.f;
                if (j < j_hi) {
#pragma unroll
                    for (int hh = 0; hh < G; ++hh)
                        lg[u][hh] = a.logit_keys ? s_logit[hh * a.logit_keys + (j - j_lo)]
                                                 : __ldcg(a.ws_s + (int64_t)(b * H + h0 + hh) * cap + j);
                    if (!(app && j == ln)) old[u] = acc[j];                  // a new entry starts at zero
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = j0 + u * kDecThreads;
                if (j < j_hi) {
                    float pr = 0.f;
#pragma unroll
                    for (int hh = 0; hh < G; ++hh) pr += exp2f(lg[u][hh] - mx[hh]) * il[hh];
                    acc[j] = old[u] + pr;
                }
            }
        }
    }
    if (app && rank == 0 && tid == 0) a.len[hd] = lne;    // every CTA of the cluster read it before the barrier
    if (CL) cluster_wait();                               // nobody leaves while its shared memory is still read
}

template <int G>
static lvlm_status launch_decode(const void* q, void* Kc, void* Vc, int32_t* len, const void* k_new,
                                 const void* v_new, float* acc_score, const lvlm_dims* d, float scale,
                                 void* out, char* wsb, const DecodeLayout& L, int64_t kv_sb,
                                 int64_t kv_sh, int32_t* dev_status, cudaStream_t stream) {
    // scaled logits of a CTA's own keys stay in shared memory when the longest run fits the budget
    const int nt_max = (d->cap + kTileKeys - 1) / kTileKeys;
    int per = (nt_max + L.S - 1) / L.S;
    if (per >= kDecWarps) per = (per + kDecWarps - 1) / kDecWarps * kDecWarps;
    const int run_keys = per * kTileKeys;
    const int logit_keys = acc_score && (size_t)G * run_keys * 4 <= (size_t)kDecLogitBytes ? run_keys : 0;
    const size_t smem = 1024 + (size_t)kRingBytes + (size_t)(2 * kDecWarps * 8 + 4 * 8 + 2 * 8 * kDecMaxCluster) * 4 +
                        (size_t)(2 * kStagesDec + 1) * 8 + (size_t)G * logit_keys * 4;
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(decode_cluster_kernel<G, true>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(decode_cluster_kernel<G, false>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    CUtensorMap kmap, vmap;
    {
        const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)d->cap, (uint64_t)d->Hkv, (uint64_t)d->B};
        const uint64_t strides[3] = {(uint64_t)kHeadDim * 2, (uint64_t)kv_sh * 2, (uint64_t)kv_sb * 2};
        const uint32_t box[4] = {64, (uint32_t)kStageKeys, 1, 1};
        if (!make_tmap_bf16(&kmap, Kc, 4, dims, strides, box) || !make_tmap_bf16(&vmap, Vc, 4, dims, strides, box))
            return LVLM_ERR_CUDA;
    }
    const int64_t ctas = (int64_t)d->B * d->Hkv * L.S;
    if (ctas > 0x7FFFFFFFll) return LVLM_ERR_UNSUPPORTED;
    DecodeArgs a;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.Kc = static_cast<__nv_bfloat16*>(Kc);
    a.Vc = static_cast<__nv_bfloat16*>(Vc);
    a.len = len;
    a.k_new = static_cast<const __nv_bfloat16*>(k_new);
    a.v_new = static_cast<const __nv_bfloat16*>(v_new);
    a.acc_score = acc_score;
    a.out = static_cast<__nv_bfloat16*>(out);
    a.H = d->H; a.Hkv = d->Hkv; a.cap = d->cap; a.S = L.S;
    a.early = d->cache_stable != 0 && pdl_enabled();
    a.kv_sb = kv_sb; a.kv_sh = kv_sh; a.scale_log2 = scale * kLog2e;
    a.ws_s = acc_score ? reinterpret_cast<float*>(wsb + L.off_s) : nullptr;
    a.logit_keys = logit_keys;
    a.dev_status = dev_status;

    if (L.S == 1)
        return launch_kernel(decode_cluster_kernel<G, false>, dim3((unsigned)ctas), dim3(kDecThreads), smem, stream, 1, kmap, vmap, a);
    return launch_kernel(decode_cluster_kernel<G, true>, dim3((unsigned)ctas), dim3(kDecThreads), smem, stream, L.S, kmap, vmap, a);
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_decode_attn(const void* q, void* Kc, void* Vc, int32_t* len,
                                         const void* k_new, const void* v_new, float* acc_score,
                                         const lvlm_dims* d, float scale, void* out, void* ws,
                                         size_t ws_bytes, int32_t* dev_status, void* stream_) {
    using namespace lvlm;
    cudaStream_t stream = (cudaStream_t)stream_;
    DecodeLayout L;
    if (!q || !Kc || !Vc || !len || !out || !decode_layout(d, &L)) return LVLM_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr)) return LVLM_ERR_INVALID_ARG;
    const int G = d->H / d->Hkv;
    if (d->D != kHeadDim || G > kMaxGroup) return LVLM_ERR_UNSUPPORTED;
    const int64_t kv_sh = d->kv_stride_h ? d->kv_stride_h : (int64_t)d->cap * d->D;
    const int64_t kv_sb = d->kv_stride_b ? d->kv_stride_b : (int64_t)d->Hkv * kv_sh;
    if (!aligned16(q) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(out) || !aligned16(k_new) ||
        !aligned16(v_new) || kv_sh % 8 || kv_sb % 8)
        return LVLM_ERR_ALIGNMENT;
    if (!ws || !aligned256(ws) || ws_bytes < L.total) return LVLM_ERR_WORKSPACE;
    char* wsb = static_cast<char*>(ws);
#define LVLM_DEC_CASE(GG)                                                                         \
    case GG: return launch_decode<GG>(q, Kc, Vc, len, k_new, v_new, acc_score, d, scale, out, wsb, \
                                      L, kv_sb, kv_sh, dev_status, stream)
    switch (G) {
        LVLM_DEC_CASE(1); LVLM_DEC_CASE(2); LVLM_DEC_CASE(3); LVLM_DEC_CASE(4);
        LVLM_DEC_CASE(5); LVLM_DEC_CASE(6); LVLM_DEC_CASE(7); LVLM_DEC_CASE(8);
    }
#undef LVLM_DEC_CASE
    return LVLM_ERR_UNSUPPORTED;
}

// ---- decode attention for callers that cannot allocate ------------------------------------------
// Scratch of lvlm_decode_attn_static: one array per GPU that loads the library, held until the
// process exits.  In host code the name below is only a handle for cudaGetSymbolAddress, never a
// pointer a kernel may be given.
static __device__ __align__(256) unsigned char g_decode_static_scratch[LVLM_STATIC_SCRATCH_BYTES];

namespace lvlm {

constexpr int kMaxStaticDevices = 64;
static void* g_static_scratch_ptr[kMaxStaticDevices];     // device address of the array, per device
static std::mutex g_static_scratch_mutex;

// Device address of the scratch array on the current device, looked up once per device.
static lvlm_status static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxStaticDevices) return LVLM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_decode_static_scratch) != cudaSuccess || !p) return LVLM_ERR_CUDA;
        g_static_scratch_ptr[dev] = p;
    }
    *out = g_static_scratch_ptr[dev];
    return LVLM_OK;
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_decode_attn_static(const void* q, void* Kc, void* Vc, int32_t* len,
                                                const void* k_new, const void* v_new,
                                                float* acc_score, const lvlm_dims* d, float scale,
                                                void* out, int32_t* dev_status, void* stream) {
    using namespace lvlm;
    DecodeLayout L;
    if (!decode_layout(d, &L)) return LVLM_ERR_INVALID_ARG;
    if (L.total > (size_t)LVLM_STATIC_SCRATCH_BYTES) return LVLM_ERR_WORKSPACE;
    void* scratch = nullptr;
    const lvlm_status st = static_scratch_address(&scratch);
    if (st != LVLM_OK) return st;
    return lvlm_decode_attn(q, Kc, Vc, len, k_new, v_new, acc_score, d, scale, out, scratch,
                            (size_t)LVLM_STATIC_SCRATCH_BYTES, dev_status, stream);
}
