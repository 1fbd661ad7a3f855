// lvlm_prefill_attn: the causal attention of a prefill layer that hands the token reduction its scores as a
// by-product (Section 3.2.1, paragraph 3 and its footnote: the per-key summed attention comes out of the
// attention kernel that runs anyway, so no separate pass over Q K^T is paid for the row normalisers).
//
// One CTA per (sequence, query head, tile of 128 query rows); tcgen05 MMAs, accumulators in tensor memory:
//   S = Q K_j^T      A = Q tile, copied once from shared into tensor memory (bf16 pairs a column), B = K tile, K-major
//                    from TMA (128-byte swizzle), 128x128 fp32 in TMEM (two buffers: the tile after next is multiplied
//                    while this one is in the softmax)
//   softmax          eight warps: thread = (query row, half of the tile's 128 keys); the row maximum of a tile meets
//                    in shared memory (one named barrier a tile); running max m and sum l in the log2 domain.  The
//                    probabilities 2^(s - m) go back into the tensor-memory columns the logits came from, as
//                    bf16 pairs (head and remainder of every probability: a plain bf16 would miss the output
//                    tolerance on rows that see few keys), so P never touches shared memory and the buffer of a
//                    tile holds first its S, then its P.  The output accumulator is rescaled only when the maximum
//                    has grown by more than 2^8 (the stale maximum keeps every probability below 2^8, well inside
//                    bf16 and fp32), and only then does the softmax wait for the product before it
//   O += P V_j       A = P from tensor memory, B = V tile as it lies in memory (keys x channels: an MN-major
//                    operand), 128x128 fp32 in TMEM; the next S is written into a buffer only when the product
//                    that read its P is complete
// At the end a thread divides its half row by l, writes it, writes lse = ln sum exp of the row, and - for the rows
// of the scoring window - the log2-domain normaliser the column-sum pass of lvlm_score_tokens reads; that pass then
// runs on the same stream (keys on the TMEM lanes, see score_tc.cu) and produces score and score_head.
#include "common.cuh"
#include "score.cuh"
#include "sm100.cuh"

namespace lvlm {

using namespace sm100;

constexpr int kAT = 128;                     // query rows per CTA, keys per tile, head dim
constexpr int kAHalf = kAT * 64 * 2;         // one TMA box: 128 rows x 64 bf16 = 16 KB
constexpr int kATile = 2 * kAHalf;           // 32 KB
constexpr int kAStages = 2;                  // K ring and V ring (released separately: K after S, V after O)
constexpr int kASoftmaxThreads = 256;        // warps 2..9
constexpr int kAThreads = 64 + kASoftmaxThreads;   // warp 0 TMA, warp 1 MMA
constexpr uint32_t kATmemCols = 512;         // S0/P0 | S1/P1 | O | Q (64 columns) | (unused)
constexpr float kLog2eA = 1.4426950408889634f;
constexpr float kLn2A = 0.6931471805599453f;
constexpr float kRescaleStep = 8.0f;         // the output is rescaled when the row maximum has grown by more (log2)

struct AttnArgs {
    int B, H, G, N, causal, q_lo, q_hi;
    float scale_log2;
    __nv_bfloat16* out; int64_t out_sb, out_sn, out_sh;   // elements
    float* lse;                // [B][H][N] natural log
    float* lse_win;            // [B][H][q_hi-q_lo] log2 domain, or NULL
    int32_t* dev_status;
};

struct AttnSmem {
    uint64_t q_full, k_full[kAStages], k_empty[kAStages], v_full[kAStages], v_empty[kAStages], s_full[2], p_ready, o_done, q_ready;
    uint32_t tmem_base;
    volatile int abort;
    float xmax[2][2][kAT];     // [tile parity][half][row]: the tile maximum of a half row, for the other half
    float xl[kAT];             // the sum of the upper half row, for the thread that writes lse
};

// D[tmem] (+)= A[tmem] * B[smem]^T, issued by one thread: A is 128 rows (lanes) of bf16 pairs, two K indices a column.
__device__ __forceinline__ void mma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// Shared-memory descriptor of an MN-major bf16 operand stored as rows of 128 bytes (64 elements of the M or N
// dimension) with the 128-byte swizzle, one row per K index: 8 rows are one swizzle atom (stride byte offset 1024
// between atoms along K), the next 64 elements of M/N start `lbo` bytes further (leading byte offset).
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr, uint32_t lbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// 32 consecutive fp32 columns of this thread's TMEM lane, written back.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
    const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ bool attn_wait(uint64_t* bar, uint32_t parity, AttnSmem* sm, int32_t* dev_status) {
    if (sm->abort) return false;
    if (mbar_wait(bar, parity)) return true;
    sm->abort = 1;
    if (dev_status) atomicOr(dev_status, LVLM_DEV_TIMEOUT);
    return false;
}

// grid (query tiles, H, B); the tiles with the most keys go first
__global__ void __launch_bounds__(kAThreads, 1)
prefill_attn_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                    const __grid_constant__ CUtensorMap vmap, const AttnArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    unsigned char* sQ = base;
    unsigned char* sK = base + kATile;                            // [kAStages] tiles
    unsigned char* sV = sK + kAStages * kATile;                   // [kAStages] tiles
    AttnSmem* sm = reinterpret_cast<AttnSmem*>(sV + kAStages * kATile);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x, h = blockIdx.y, b = blockIdx.z, g = h / a.G;
    const int row_end = min(a.N, (qt + 1) * kAT);                // one past the last valid query of the tile
    const int key_end = a.causal ? row_end : a.N;                // keys this tile can see
    const int nk = (key_end + kAT - 1) / kAT;

    if (threadIdx.x == 0) {
        mbar_init(&sm->q_full, 1);
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(&sm->k_full[s], 1); mbar_init(&sm->k_empty[s], 1);
            mbar_init(&sm->v_full[s], 1); mbar_init(&sm->v_empty[s], 1);
        }
        for (int s = 0; s < 2; ++s) mbar_init(&sm->s_full[s], 1);
        mbar_init(&sm->p_ready, kASoftmaxThreads);
        mbar_init(&sm->o_done, 1);
        mbar_init(&sm->q_ready, kAT);
        sm->abort = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&qmap);
        prefetch_tmap(&kmap);
        prefetch_tmap(&vmap);
    }
    if (warp == 1) tmem_alloc(&sm->tmem_base, kATmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    const uint32_t tmem_o = tmem_base + 2 * kAT;
    const uint32_t tmem_q = tmem_base + 3 * kAT;
    pdl_enter();

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            mbar_arrive_expect_tx(&sm->q_full, kATile);
            tma_load_4d(sQ, &qmap, &sm->q_full, 0, h, qt * kAT, b);
            tma_load_4d(sQ + kAHalf, &qmap, &sm->q_full, 64, h, qt * kAT, b);
            for (int j = 0; j < nk; ++j) {
                const int st = j % kAStages;
                if (j >= kAStages && !attn_wait(&sm->k_empty[st], ((j / kAStages) - 1) & 1, sm, a.dev_status)) break;
                mbar_arrive_expect_tx(&sm->k_full[st], kATile);
                tma_load_4d(sK + st * kATile, &kmap, &sm->k_full[st], 0, j * kAT, g, b);
                tma_load_4d(sK + st * kATile + kAHalf, &kmap, &sm->k_full[st], 64, j * kAT, g, b);
                if (j >= kAStages && !attn_wait(&sm->v_empty[st], ((j / kAStages) - 1) & 1, sm, a.dev_status)) break;
                mbar_arrive_expect_tx(&sm->v_full[st], kATile);
                tma_load_4d(sV + st * kATile, &vmap, &sm->v_full[st], 0, j * kAT, g, b);
                tma_load_4d(sV + st * kATile + kAHalf, &vmap, &sm->v_full[st], 64, j * kAT, g, b);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        // The whole warp runs the loop (same values in every lane, so that they can live in uniform registers); one
        // elected lane issues the MMAs and the commits.
        {
            constexpr uint32_t idesc_qk = idesc_bf16_f32(kAT, kAT);
            constexpr uint32_t idesc_pv = idesc_bf16_f32(kAT, kAT) | (1u << 16);     // B (the V tile) is MN-major
            // S_j into buffer j & 1, over P_{j-2} (the caller has waited for the product that read it)
            // (this thread shares its scheduler with two softmax warps: whatever an MMA needs is worked out before the
            // wait, so that the MMAs themselves go out back to back)
            auto issue_qk = [&](int j) -> bool {
                const int st = j % kAStages;
                const uint32_t k_addr = smem_u32(sK + st * kATile);
                const uint32_t d_tmem = tmem_base + (j & 1) * kAT;
                uint64_t kd[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) kd[k] = smem_desc_sw128(k_addr + (k >> 2) * kAHalf + (k & 3) * 32);
                if (!__all_sync(0xFFFFFFFFu, attn_wait(&sm->k_full[st], (j / kAStages) & 1, sm, a.dev_status))) return false;
                tc_fence_after();
                if (elect_one()) {
                    mma_bf16_ts(d_tmem, tmem_q, kd[0], idesc_qk, 0u);       // 16 channels per step: 8 columns of bf16 pairs
#pragma unroll
                    for (int k = 1; k < 8; ++k) mma_bf16_ts(d_tmem, tmem_q + k * 8, kd[k], idesc_qk, 1u);
                    mma_commit(&sm->k_empty[st]);              // the K tile may be refilled once these are done
                    mma_commit(&sm->s_full[j & 1]);
                }
                __syncwarp();
                return true;
            };
            bool ok = __all_sync(0xFFFFFFFFu, attn_wait(&sm->q_ready, 0, sm, a.dev_status));
            if (ok && nk > 0) ok = issue_qk(0);
            if (ok && nk > 1) ok = issue_qk(1);
            for (int j = 0; ok && j < nk; ++j) {
                const uint32_t v_addr = smem_u32(sV + (j % kAStages) * kATile);
                const uint32_t p_tmem = tmem_base + (j & 1) * kAT;
                uint64_t vd[8];                             // 16 keys per step: 8 columns of bf16 pairs
#pragma unroll
                for (int k = 0; k < 8; ++k) vd[k] = smem_desc_mn_sw128(v_addr + k * 2048, kAHalf);
                ok = attn_wait(&sm->v_full[j % kAStages], (j / kAStages) & 1, sm, a.dev_status);
                if (ok) ok = attn_wait(&sm->p_ready, j & 1, sm, a.dev_status);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    mma_bf16_ts(tmem_o, p_tmem, vd[0], idesc_pv, j > 0 ? 1u : 0u);       // heads; the remainders lie 16 columns on
                    mma_bf16_ts(tmem_o, p_tmem + 16, vd[0], idesc_pv, 1u);
#pragma unroll
                    for (int k = 1; k < 8; ++k) {
                        const uint32_t pa = p_tmem + (k >> 1) * 32 + (k & 1) * 8;
                        mma_bf16_ts(tmem_o, pa, vd[k], idesc_pv, 1u);
                        mma_bf16_ts(tmem_o, pa + 16, vd[k], idesc_pv, 1u);
                    }
                    mma_commit(&sm->v_empty[j % kAStages]);     // the V tile is done with
                    mma_commit(&sm->o_done);
                }
                __syncwarp();
                if (j + 2 < nk) {
                    // The logits of the tile after next go where this tile's P lies: not before the product has read it
                    // (the softmax of the next tile is far from done by then, so nothing waits for this wait).
                    ok = __all_sync(0xFFFFFFFFu, attn_wait(&sm->o_done, j & 1, sm, a.dev_status));
                    if (ok) ok = issue_qk(j + 2);
                }
            }
        }
    } else {
        // ================= softmax: thread = (query row, half of the keys of a tile) =================
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const int pos = qt * kAT + row;                      // sequence position of my query
        const uint32_t lane_addr = ((uint32_t)(quarter * 32) << 16);
        float m_used = -INFINITY, l_run = 0.f;               // l_run: the sum over my half of the keys
        // The Q tile goes from shared memory into tensor memory once (thread = row, bf16 pairs a column): S = Q K^T
        // then reads only K from shared memory, which is what lets these MMAs run at the pace of the pipe.
        if (half == 0) {
            const bool got = __all_sync(0xFFFFFFFFu, attn_wait(&sm->q_full, 0, sm, a.dev_status));
            if (got) {
#pragma unroll
                for (int hq = 0; hq < 2; ++hq) {             // 64 channels = 32 columns
                    uint32_t w[32];
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        const uint4 x = *reinterpret_cast<const uint4*>(sQ + hq * kAHalf + row * 128 + ((ch ^ (row & 7)) << 4));
                        w[4 * ch] = x.x; w[4 * ch + 1] = x.y; w[4 * ch + 2] = x.z; w[4 * ch + 3] = x.w;
                    }
                    tmem_st32(tmem_q + lane_addr + hq * 32, reinterpret_cast<const float*>(w));
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&sm->q_ready);
            }
        }
        // Every thread runs every round and meets the others at the named barrier, also after a wait has given up
        // (`ok`, the same for all lanes of a warp, then only switches the work off).
        bool ok = true;
        for (int j = 0; j < nk; ++j) {
            const int buf = j & 1;
            ok = __all_sync(0xFFFFFFFFu, ok && attn_wait(&sm->s_full[buf], (j / 2) & 1, sm, a.dev_status));
            const uint32_t s_addr = tmem_base + lane_addr + buf * kAT + half * 64;
            const int lim = min(a.N, a.causal ? pos + 1 : a.N) - j * kAT - half * 64;   // my columns c < lim are visible
            float v[2][32];
            float tmax = -INFINITY;
            // off the diagonal every lane of the warp sees all of its 64 keys: no masks then
            const bool full = __all_sync(0xFFFFFFFFu, lim >= 64);
            if (ok) {
                tc_fence_after();
                tmem_ld32(s_addr, v[0]);
                tmem_ld32(s_addr + 32, v[1]);
                tmem_ld_wait();
                if (full) {
                    float t0 = v[0][0], t1 = v[0][1], t2 = v[1][0], t3 = v[1][1];
#pragma unroll
                    for (int c = 2; c < 32; c += 2) {
                        t0 = fmaxf(t0, v[0][c]); t1 = fmaxf(t1, v[0][c + 1]);
                        t2 = fmaxf(t2, v[1][c]); t3 = fmaxf(t3, v[1][c + 1]);
                    }
                    tmax = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3));
                } else {
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2)
#pragma unroll
                        for (int c = 0; c < 32; ++c) tmax = fmaxf(tmax, c2 * 32 + c < lim ? v[c2][c] : -INFINITY);
                }
            }
            // the maximum of the row's other half
            sm->xmax[buf][half][row] = tmax;
            asm volatile("bar.sync 1, %0;" ::"n"(kASoftmaxThreads) : "memory");
            if (!ok) continue;
            tmax = fmaxf(tmax, sm->xmax[buf][half ^ 1][row]);
            tmax *= a.scale_log2;                            // a positive scale keeps the order
            float corr = 1.f;
            bool grow = false;
            if (tmax > -INFINITY && (m_used == -INFINITY || tmax > m_used + kRescaleStep)) {
                corr = m_used == -INFINITY ? 0.f : ex2_approx(m_used - tmax);
                m_used = tmax;
                grow = true;
            }
            // O is touched only when some row of the warp moves its reference: the products issued so far have to be done
            if (j > 0 && __any_sync(0xFFFFFFFFu, grow)) {
                ok = __all_sync(0xFFFFFFFFu, attn_wait(&sm->o_done, (j - 1) & 1, sm, a.dev_status));
                if (!ok) continue;
                tc_fence_after();
                l_run *= corr;
#pragma unroll 1
                for (int c2 = 0; c2 < 2; ++c2) {             // my half of the channels
                    float o[32];
                    tmem_ld32(tmem_o + lane_addr + half * 64 + c2 * 32, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c] *= corr;
                    tmem_st32(tmem_o + lane_addr + half * 64 + c2 * 32, o);
                }
                tmem_st_wait();
            }
            // probabilities relative to m_used, written over the logits they came from: 32 logits become 16 columns
            // of bf16 pairs (the bf16 rounding of every probability) and 16 columns of what the rounding left
            const float mref = m_used == -INFINITY ? 0.f : m_used;
            float psum = 0.f;
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    float p0 = ex2_approx(fmaf(v[c2][c], a.scale_log2, -mref));
                    float p1 = ex2_approx(fmaf(v[c2][c + 1], a.scale_log2, -mref));
                    if (!full) {
                        p0 = c2 * 32 + c < lim ? p0 : 0.f;
                        p1 = c2 * 32 + c + 1 < lim ? p1 : 0.f;
                    }
                    pk[c >> 1] = pack_bf16(p0, p1);
                    pk[16 + (c >> 1)] = pack_bf16(p0 - bf16_lo(pk[c >> 1]), p1 - bf16_hi(pk[c >> 1]));
                    psum += p0 + p1;
                }
                tmem_st32(s_addr + c2 * 32, reinterpret_cast<const float*>(pk));
            }
            l_run += psum;
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&sm->p_ready);
        }
        // ---- the output row --------------------------------------------------------------------------------
        ok = __all_sync(0xFFFFFFFFu, ok && (nk == 0 || attn_wait(&sm->o_done, (nk - 1) & 1, sm, a.dev_status)));
        tc_fence_after();
        if (half == 1) sm->xl[row] = l_run;
        asm volatile("bar.sync 1, %0;" ::"n"(kASoftmaxThreads) : "memory");
        {
            const float l_row = half == 0 ? l_run + sm->xl[row] : 0.f;
            if (half == 0) sm->xl[row] = l_row;
            asm volatile("bar.sync 1, %0;" ::"n"(kASoftmaxThreads) : "memory");
            const float l_all = sm->xl[row];
            const bool valid = ok && pos < a.N && !sm->abort;
            const float inv = l_all > 0.f ? 1.0f / l_all : 0.f;
            __nv_bfloat16* orow = a.out + (int64_t)b * a.out_sb + (int64_t)pos * a.out_sn + (int64_t)h * a.out_sh + half * 64;
#pragma unroll 1
            for (int c2 = 0; c2 < 2; ++c2) {                // (the loads are warp-wide: every lane takes part)
                float o[32];
                tmem_ld32(tmem_o + lane_addr + half * 64 + c2 * 32, o);
                tmem_ld_wait();
                if (valid) {
                    uint4* dst = reinterpret_cast<uint4*>(orow + c2 * 32);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        dst[q] = make_uint4(pack_bf16(o[8 * q] * inv, o[8 * q + 1] * inv), pack_bf16(o[8 * q + 2] * inv, o[8 * q + 3] * inv),
                                            pack_bf16(o[8 * q + 4] * inv, o[8 * q + 5] * inv), pack_bf16(o[8 * q + 6] * inv, o[8 * q + 7] * inv));
                }
            }
            if (valid && half == 0) {
                const float lse2 = m_used + log2f(l_all);   // log2 of the row's sum of 2^(scaled logits)
                a.lse[((int64_t)b * a.H + h) * a.N + pos] = lse2 * kLn2A;
                if (a.lse_win && pos >= a.q_lo && pos < a.q_hi)
                    a.lse_win[((int64_t)b * a.H + h) * (a.q_hi - a.q_lo) + (pos - a.q_lo)] = lse2;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (sm->abort) {                              // let copies still in flight land before leaving
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kATmemCols);
    }
}

size_t prefill_attn_workspace(const lvlm_dims* d) {
    ScoreLayout L;
    return score_layout(d, &L) ? L.total : 0;
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_prefill_attn(const void* Q, const void* K, const void* V, const lvlm_dims* d,
                                          float scale, void* out, float* lse, float* score, float* score_head,
                                          void* ws, size_t ws_bytes, int32_t* dev_status, void* stream_) {
    using namespace lvlm;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!Q || !K || !V || !out || !lse || !d || d->B <= 0 || d->H <= 0 || d->Hkv <= 0 || d->H % d->Hkv || d->N <= 0 ||
        d->cap < d->N || !(scale > 0.f))
        return LVLM_ERR_INVALID_ARG;
    if (score_head && !score) return LVLM_ERR_INVALID_ARG;
    if (d->D != kHeadDim) return LVLM_ERR_UNSUPPORTED;
    ScoreLayout L;
    if (score && !score_layout(d, &L)) return LVLM_ERR_INVALID_ARG;
    if (score && d->head_stride != 0 && d->head_stride < d->n) return LVLM_ERR_INVALID_ARG;
    ScoreStrides st;
    st.q_sh = d->q_stride_h ? d->q_stride_h : d->D;
    st.q_sn = d->q_stride_n ? d->q_stride_n : (int64_t)d->H * d->D;
    st.q_sb = d->q_stride_b ? d->q_stride_b : (int64_t)d->N * st.q_sn;
    st.kv_sh = d->kv_stride_h ? d->kv_stride_h : (int64_t)d->cap * d->D;
    st.kv_sb = d->kv_stride_b ? d->kv_stride_b : (int64_t)d->Hkv * st.kv_sh;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(out) || st.q_sh % 8 || st.q_sn % 8 || st.q_sb % 8 ||
        st.kv_sh % 8 || st.kv_sb % 8)
        return LVLM_ERR_ALIGNMENT;
    char* wsb = static_cast<char*>(ws);
    if (score && (!ws || !aligned256(ws) || ws_bytes < L.total)) return LVLM_ERR_WORKSPACE;

    CUtensorMap qmap, kmap, vmap;
    {
        const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)d->H, (uint64_t)d->N, (uint64_t)d->B};
        const uint64_t strides[3] = {(uint64_t)st.q_sh * 2, (uint64_t)st.q_sn * 2, (uint64_t)st.q_sb * 2};
        const uint32_t box[4] = {64, 1, (uint32_t)kAT, 1};
        if (!make_tmap_bf16(&qmap, Q, 4, dims, strides, box)) return LVLM_ERR_CUDA;
    }
    {
        const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)d->N, (uint64_t)d->Hkv, (uint64_t)d->B};
        const uint64_t strides[3] = {(uint64_t)kHeadDim * 2, (uint64_t)st.kv_sh * 2, (uint64_t)st.kv_sb * 2};
        const uint32_t box[4] = {64, (uint32_t)kAT, 1, 1};
        if (!make_tmap_bf16(&kmap, K, 4, dims, strides, box) || !make_tmap_bf16(&vmap, V, 4, dims, strides, box))
            return LVLM_ERR_CUDA;
    }
    AttnArgs a;
    a.B = d->B; a.H = d->H; a.G = d->H / d->Hkv; a.N = d->N; a.causal = d->causal;
    a.q_lo = score ? d->q_lo : 0; a.q_hi = score ? d->q_hi : 0;
    a.scale_log2 = scale * kLog2eA;
    a.out = static_cast<__nv_bfloat16*>(out);
    a.out_sh = d->D; a.out_sn = (int64_t)d->H * d->D; a.out_sb = (int64_t)d->N * a.out_sn;
    a.lse = lse;
    a.lse_win = score ? reinterpret_cast<float*>(wsb + L.off_lse) : nullptr;
    a.dev_status = dev_status;
    const size_t smem = 1024 + (size_t)kATile * (1 + 2 * kAStages) + sizeof(AttnSmem);
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(prefill_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int nqt = (d->N + kAT - 1) / kAT;
    lvlm_status s0 = launch_kernel(prefill_attn_kernel, dim3(nqt, d->H, d->B), dim3(kAThreads), smem, stream, 1,
                                   qmap, kmap, vmap, a);
    if (s0 != LVLM_OK || !score) return s0;
    // the column sums of the window: the second pass of lvlm_score_tokens, fed by the normalisers written above
    const __nv_bfloat16* Qwin = static_cast<const __nv_bfloat16*>(Q) + (int64_t)d->q_lo * st.q_sn;
    return launch_score_tc(Qwin, K, nullptr, d, st, scale, reinterpret_cast<float*>(wsb + L.off_lse),
                           reinterpret_cast<float*>(wsb + L.off_partial), reinterpret_cast<int32_t*>(wsb + L.off_cnt),
                           score, score_head, dev_status, stream, /*normalisers_ready=*/true);
}
