// lvlm_decode_attn: one generated token attends to every cached key and value of its KV head
// (Section 3.2.2, paragraph 1), over caches whose lengths differ per (sequence, KV head) after
// compression.  HBM-bound: every K and V row is read once and shared by the G query heads of
// the group.
//
// Split-K: grid (splits, Hkv, B).  Inside a CTA every warp streams its own 16-key tiles through a
// private ring of shared-memory stages (cp.async, 16-byte chunks XOR-swizzled so that ldmatrix is
// conflict free), multiplies them with small tensor-core MMAs (the G query heads of the group are
// the rows of a 16-row tile) and keeps an online softmax per head, so the main loop has no block
// barrier.  The four warps' (max, sum, output) are merged once at the end and parked per split; a
// second kernel combines the splits in split order, writes bf16 outputs, adds the group-summed
// probabilities to acc_score and bumps len after an append.
#include <mutex>

#include "common.cuh"

namespace lvlm {

constexpr int kDecThreads = 128;
constexpr int kDecWarps = 4;
constexpr int kTileKeys = 16;                        // keys per warp tile
constexpr int kStagesDec = 3;                        // stages per warp
constexpr int kTileHalf = kTileKeys * 256;           // bytes of one K (or V) tile
constexpr int kStageBytes = 2 * kTileHalf;           // K tile then V tile
constexpr float kLog2e = 1.4426950408889634f;

struct DecodeLayout { int chunk, nsplit; size_t off_o, off_ml, off_s, total; };

static bool decode_layout(const lvlm_dims* d, DecodeLayout* L) {
    if (!d || d->B <= 0 || d->H <= 0 || d->Hkv <= 0 || d->H % d->Hkv || d->cap <= 0) return false;
    // as many CTAs as fit on the GPU at once (two per SM), chunks a multiple of 64 keys so that
    // every warp of a CTA has at least one tile
    const int heads = d->B * d->Hkv;
    int want = (2 * 148 + heads - 1) / heads;
    if (want < 1) want = 1;
    int chunk = (d->cap + want - 1) / want;
    chunk = (chunk + 63) / 64 * 64;
    L->chunk = chunk;
    L->nsplit = (d->cap + chunk - 1) / chunk;
    size_t off = 0;
    const size_t bh = (size_t)d->B * d->H;
    L->off_o = off;  off = align_up(off + bh * L->nsplit * kHeadDim * 4, 256);
    L->off_ml = off; off = align_up(off + bh * L->nsplit * 2 * 4, 256);
    L->off_s = off;  off = align_up(off + bh * d->cap * 4, 256);
    L->total = off;
    return true;
}

size_t decode_attn_workspace(const lvlm_dims* d) {
    DecodeLayout L;
    return decode_layout(d, &L) ? L.total : 0;
}

// 16-byte asynchronous copy; src_bytes = 0 writes zeros instead.
__device__ __forceinline__ void cp_async16_zfill(uint32_t smem, const void* gmem, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem), "l"(gmem), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

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

template <int G>
__global__ void __launch_bounds__(kDecThreads, 2)
decode_split_kernel(const __nv_bfloat16* __restrict__ q, __nv_bfloat16* Kc, __nv_bfloat16* Vc,
                    const int32_t* __restrict__ len, const __nv_bfloat16* __restrict__ k_new,
                    const __nv_bfloat16* __restrict__ v_new, int H, int Hkv, int cap,
                    int64_t kv_sb, int64_t kv_sh, float scale_log2, int chunk, int nsplit,
                    float* __restrict__ ws_o, float* __restrict__ ws_ml, float* __restrict__ ws_s,
                    int want_logits, int32_t* dev_status) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int hd = b * Hkv + g;
    int ln = len[hd];
    if (ln < 0 || ln > cap) {                         // corrupt length: treat the head as empty
        if (tid == 0 && dev_status) atomicOr(dev_status, LVLM_DEV_BOUNDS);
        ln = 0;
    }
    const bool append = k_new != nullptr && ln < cap;
    if (k_new != nullptr && ln >= cap && tid == 0 && split == 0 && dev_status)
        atomicOr(dev_status, LVLM_DEV_BOUNDS);
    const int ln_eff = ln + (append ? 1 : 0);
    const int j_begin = split * chunk;
    const int j_end = min(ln_eff, j_begin + chunk);
    const int h0 = g * G;

    float* my_o = ws_o + ((int64_t)(b * H + h0) * nsplit + split) * kHeadDim;      // + hh*nsplit*128
    float* my_ml = ws_ml + ((int64_t)(b * H + h0) * nsplit + split) * 2;           // + hh*nsplit*2
    if (j_begin >= j_end) {
        if (tid < G) { my_ml[(int64_t)tid * nsplit * 2] = -INFINITY; my_ml[(int64_t)tid * nsplit * 2 + 1] = 0.f; }
        return;
    }
    __nv_bfloat16* Kseq = Kc + (int64_t)b * kv_sb + (int64_t)g * kv_sh;
    __nv_bfloat16* Vseq = Vc + (int64_t)b * kv_sb + (int64_t)g * kv_sh;
    const __nv_bfloat16* kn = append ? k_new + (int64_t)hd * kHeadDim : nullptr;
    const __nv_bfloat16* vn = append ? v_new + (int64_t)hd * kHeadDim : nullptr;

    // the CTA whose chunk holds row `ln` stores the appended row into the cache
    if (append && ln >= j_begin && ln < j_end && tid < 32) {
        const uint2 kv = reinterpret_cast<const uint2*>(kn)[lane];
        const uint2 vv = reinterpret_cast<const uint2*>(vn)[lane];
        reinterpret_cast<uint2*>(Kseq + (int64_t)ln * kHeadDim)[lane] = kv;
        reinterpret_cast<uint2*>(Vseq + (int64_t)ln * kHeadDim)[lane] = vv;
    }

    // ---- query fragments: heads of the group are rows 0..G-1 of a 16-row A tile -------------------
    const int row = lane >> 2, qd = lane & 3;
    uint32_t qa[8][2];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        qa[ks][0] = qa[ks][1] = 0u;
        if (row < G) {
            const uint32_t* qp = reinterpret_cast<const uint32_t*>(q + (int64_t)(b * H + h0 + row) * kHeadDim);
            qa[ks][0] = __ldg(qp + ks * 8 + qd);
            qa[ks][1] = __ldg(qp + ks * 8 + 4 + qd);
        }
    }

    // ---- per-warp tile ring --------------------------------------------------------------------------
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(smem) + warp * (kStagesDec * kStageBytes);
    const int ntile_cta = (j_end - j_begin + kTileKeys - 1) / kTileKeys;
    const int my_ntile = ntile_cta > warp ? (ntile_cta - warp + kDecWarps - 1) / kDecWarps : 0;

    auto issue = [&](int it) {                 // my it-th tile -> stage it % kStagesDec
        const uint32_t st = ring + (it % kStagesDec) * kStageBytes;
        const int j0 = j_begin + (warp + it * kDecWarps) * kTileKeys;
        // 16 rows x 16 chunks per tensor = 256 chunks, 8 per lane per tensor
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int e = u * 32 + lane;
            const int r = e >> 4, c = e & 15;
            const int j = j0 + r;
            const bool ok = j < j_end;
            const bool fresh = append && j == ln;
            const __nv_bfloat16* ksrc = fresh ? kn : Kseq + (int64_t)(ok ? j : j_begin) * kHeadDim;
            const __nv_bfloat16* vsrc = fresh ? vn : Vseq + (int64_t)(ok ? j : j_begin) * kHeadDim;
            const uint32_t off = r * 256 + ((c ^ (r & 7)) << 4);
            cp_async16_zfill(st + off, ksrc + c * 8, ok ? 16 : 0);
            cp_async16_zfill(st + kTileHalf + off, vsrc + c * 8, ok ? 16 : 0);
        }
    };
#pragma unroll
    for (int it = 0; it < kStagesDec - 1; ++it) {
        if (it < my_ntile) issue(it);
        cp_async_commit();
    }

    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;      // of head `row`; l_run is this lane's share of the sum

    for (int it = 0; it < my_ntile; ++it) {
        cp_async_wait<kStagesDec - 2>();
        __syncwarp();
        const uint32_t st = ring + (it % kStagesDec) * kStageBytes;
        const int j0 = j_begin + (warp + it * kDecWarps) * kTileKeys;
        // ---- S = Q K^T for 16 keys --------------------------------------------------------------
        float s[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
        {
            const int mi = lane >> 3, r8 = lane & 7;
            const int key = (mi >> 1) * 8 + r8;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const int chunkc = 2 * ks + (mi & 1);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(st + key * 256 + ((chunkc ^ (key & 7)) << 4), b0, b1, b2, b3);
                mma_16816(s[0], qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
                mma_16816(s[1], qa[ks][0], 0u, qa[ks][1], 0u, b2, b3);
            }
        }
        // ---- online softmax of head `row` over the tile's keys --------------------------------------
        float tmax = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int j = j0 + nt * 8 + qd * 2 + c;
                float v = s[nt][c] * scale_log2;
                if (j >= j_end) v = -INFINITY;
                s[nt][c] = v;
                tmax = fmaxf(tmax, v);
                if (want_logits && row < G && j < j_end)
                    ws_s[(int64_t)(b * H + h0 + row) * cap + j] = v;
            }
        tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, 2));
        const float m_new = fmaxf(m_run, tmax);          // finite: every tile has a valid key
        const float corr = exp2f(m_run - m_new);
        m_run = m_new;
        float p[2][2];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int c = 0; c < 2; ++c) p[nt][c] = exp2f(s[nt][c] - m_new);
        l_run = l_run * corr + (p[0][0] + p[0][1]) + (p[1][0] + p[1][1]);
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) { o[nt][0] *= corr; o[nt][1] *= corr; }
        // ---- O += P V ---------------------------------------------------------------------------------
        // P is split into a bf16 head and a bf16 remainder so that the product keeps ~16 bits
        const uint32_t pa0 = pack_bf16(p[0][0], p[0][1]), pa2 = pack_bf16(p[1][0], p[1][1]);
        const uint32_t pr0 = pack_bf16(p[0][0] - bf16_lo(pa0), p[0][1] - bf16_hi(pa0));
        const uint32_t pr2 = pack_bf16(p[1][0] - bf16_lo(pa2), p[1][1] - bf16_hi(pa2));
        {
            const int mi = lane >> 3, r8 = lane & 7;
            const int key = (mi & 1) * 8 + r8;
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                const int chunkc = 2 * dp + (mi >> 1);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(st + kTileHalf + key * 256 + ((chunkc ^ (key & 7)) << 4), b0, b1, b2, b3);
                mma_16816(o[2 * dp], pa0, 0u, pa2, 0u, b0, b1);
                mma_16816(o[2 * dp + 1], pa0, 0u, pa2, 0u, b2, b3);
                mma_16816(o[2 * dp], pr0, 0u, pr2, 0u, b0, b1);
                mma_16816(o[2 * dp + 1], pr0, 0u, pr2, 0u, b2, b3);
            }
        }
        __syncwarp();
        if (it + kStagesDec - 1 < my_ntile) issue(it + kStagesDec - 1);
        cp_async_commit();
    }
    cp_async_wait<0>();
    // ---- merge the four warps, park the split's result ------------------------------------------------
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
    __syncthreads();                                       // every warp is done with its ring
    float* wm = reinterpret_cast<float*>(smem);            // [4][8]
    float* wl = wm + kDecWarps * 8;                        // [4][8]
    float* wo = wl + kDecWarps * 8;                        // [4][G][128]
    if (row < G) {
        if (qd == 0) { wm[warp * 8 + row] = m_run; wl[warp * 8 + row] = l_run; }
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
            *reinterpret_cast<float2*>(wo + ((warp * G + row) * kHeadDim) + nt * 8 + qd * 2) =
                make_float2(o[nt][0], o[nt][1]);
    }
    __syncthreads();
    for (int i = tid; i < G * kHeadDim; i += kDecThreads) {
        const int hh = i / kHeadDim, dd = i % kHeadDim;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, wm[w * 8 + hh]);
        float v = 0.f, lsum = 0.f;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) {
            const float mw = wm[w * 8 + hh];
            if (mw > -INFINITY) {
                const float f = exp2f(mw - M);
                v += wo[(w * G + hh) * kHeadDim + dd] * f;
                lsum += wl[w * 8 + hh] * f;
            }
        }
        my_o[(int64_t)hh * nsplit * kHeadDim + dd] = v;
        if (dd == 0) {
            my_ml[(int64_t)hh * nsplit * 2] = M;
            my_ml[(int64_t)hh * nsplit * 2 + 1] = lsum;
        }
    }
}

template <int G>
__global__ void __launch_bounds__(kDecThreads)
decode_combine_kernel(int32_t* len, int has_append, float* acc_score, int H, int Hkv, int cap,
                      int nsplit, const float* __restrict__ ws_o, const float* __restrict__ ws_ml,
                      const float* __restrict__ ws_s, __nv_bfloat16* __restrict__ out) {
    extern __shared__ float cw[];                  // [G][nsplit] weight of every split's partial output
    __shared__ float sM[G], sInvL[G];
    const int g = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int hd = b * Hkv + g;
    int ln = len[hd];
    if (ln < 0 || ln > cap) ln = 0;
    const bool append = has_append && ln < cap;
    const int ln_eff = ln + (append ? 1 : 0);
    const int h0 = g * G;
    const float* ml0 = ws_ml + (int64_t)(b * H + h0) * nsplit * 2;
    // all (max, sum) pairs land in shared memory with independent loads
    float* sml = cw + G * nsplit;                  // [G][nsplit][2]
    for (int i = tid; i < G * nsplit * 2; i += kDecThreads) sml[i] = ml0[i];
    __syncthreads();
    if (tid < G) {
        float M = -INFINITY;
        for (int s = 0; s < nsplit; ++s) M = fmaxf(M, sml[(tid * nsplit + s) * 2]);
        float Lsum = 0.f;
        for (int s = 0; s < nsplit; ++s) {
            const float l = sml[(tid * nsplit + s) * 2 + 1];
            const float f = l > 0.f ? exp2f(sml[(tid * nsplit + s) * 2] - M) : 0.f;
            cw[tid * nsplit + s] = f;
            Lsum += l * f;                          // split order: fixed
        }
        const float inv = Lsum > 0.f ? 1.0f / Lsum : 0.f;
        sM[tid] = M;
        sInvL[tid] = inv;
    }
    __syncthreads();
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
        const float* po = ws_o + (int64_t)(b * H + h0 + hh) * nsplit * kHeadDim + tid;
        float v = 0.f;
        int s = 0;
        for (; s + 3 < nsplit; s += 4) {
            const float w0 = cw[hh * nsplit + s], w1 = cw[hh * nsplit + s + 1];
            const float w2 = cw[hh * nsplit + s + 2], w3 = cw[hh * nsplit + s + 3];
            const float x0 = w0 != 0.f ? po[(s + 0) * kHeadDim] : 0.f;
            const float x1 = w1 != 0.f ? po[(s + 1) * kHeadDim] : 0.f;
            const float x2 = w2 != 0.f ? po[(s + 2) * kHeadDim] : 0.f;
            const float x3 = w3 != 0.f ? po[(s + 3) * kHeadDim] : 0.f;
            v += x0 * w0; v += x1 * w1; v += x2 * w2; v += x3 * w3;
        }
        for (; s < nsplit; ++s) {
            const float w0 = cw[hh * nsplit + s];
            if (w0 != 0.f) v += po[s * kHeadDim] * w0;
        }
        out[(int64_t)(b * H + h0 + hh) * kHeadDim + tid] = __float2bfloat16_rn(v * sInvL[hh]);
    }
    if (acc_score) {
        float* acc = acc_score + (int64_t)hd * cap;
        for (int j = tid; j < ln_eff; j += kDecThreads) {
            float lg[G];
#pragma unroll
            for (int hh = 0; hh < G; ++hh) lg[hh] = ws_s[(int64_t)(b * H + h0 + hh) * cap + j];
            const float old = (append && j == ln) ? 0.f : acc[j];     // a new entry starts at zero
            float p = 0.f;
#pragma unroll
            for (int hh = 0; hh < G; ++hh) p += exp2f(lg[hh] - sM[hh]) * sInvL[hh];
            acc[j] = old + p;
        }
    }
    if (append && tid == 0) len[hd] = ln_eff;
}

template <int G>
static lvlm_status launch_decode(const void* q, void* Kc, void* Vc, int32_t* len, const void* k_new,
                                 const void* v_new, float* acc_score, const lvlm_dims* d, float scale,
                                 void* out, char* wsb, const DecodeLayout& L, int64_t kv_sb,
                                 int64_t kv_sh, int32_t* dev_status, cudaStream_t stream) {
    float* ws_o = reinterpret_cast<float*>(wsb + L.off_o);
    float* ws_ml = reinterpret_cast<float*>(wsb + L.off_ml);
    float* ws_s = reinterpret_cast<float*>(wsb + L.off_s);
    size_t smem = (size_t)kDecWarps * kStagesDec * kStageBytes;
    const size_t red = (size_t)(2 * kDecWarps * 8 + kDecWarps * G * kHeadDim) * 4;
    if (red > smem) smem = red;
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(decode_split_kernel<G>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_split_kernel<G><<<dim3(L.nsplit, d->Hkv, d->B), kDecThreads, smem, stream>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(Kc),
        static_cast<__nv_bfloat16*>(Vc), len, static_cast<const __nv_bfloat16*>(k_new),
        static_cast<const __nv_bfloat16*>(v_new), d->H, d->Hkv, d->cap, kv_sb, kv_sh,
        scale * kLog2e, L.chunk, L.nsplit, ws_o, ws_ml, ws_s, acc_score != nullptr, dev_status);
    if (cudaGetLastError() != cudaSuccess) return LVLM_ERR_CUDA;
    decode_combine_kernel<G><<<dim3(d->Hkv, d->B), kDecThreads, (size_t)G * L.nsplit * 3 * 4, stream>>>(
        len, k_new != nullptr, acc_score, d->H, d->Hkv, d->cap, L.nsplit, ws_o, ws_ml, ws_s,
        static_cast<__nv_bfloat16*>(out));
    return launch_status();
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
