// lvlm_decode_attn: one generated token attends to every cached key and value of its KV head
// (Section 3.2.2, paragraph 1), over caches whose lengths differ per (sequence, KV head) after
// compression.  HBM-bound: every K and V row is read once and shared by the G query heads of
// the group.  Split-K: grid (splits, Hkv, B); each CTA streams a chunk of rows through shared
// memory (cp.async, two tiles in flight), keeps an online softmax per head and parks
// (max, sum, unnormalised output); a second kernel combines the splits in split order, writes
// bf16 outputs, adds the group-summed probabilities to acc_score and bumps len after an append.
#include "common.cuh"

namespace lvlm {

constexpr int kDecThreads = 128;
constexpr int kDecTile = 64;                         // keys per shared-memory tile
constexpr int kRowPad = 272;                         // bytes per staged row: 256 + 16 (bank spread)
constexpr float kLog2e = 1.4426950408889634f;

struct DecodeLayout { int chunk, nsplit; size_t off_o, off_ml, off_s, total; };

static bool decode_layout(const lvlm_dims* d, DecodeLayout* L) {
    if (!d || d->B <= 0 || d->H <= 0 || d->Hkv <= 0 || d->H % d->Hkv || d->cap <= 0) return false;
    // enough CTAs for a few per SM, chunks a multiple of the tile
    const int heads = d->B * d->Hkv;
    int want = (4 * 148 + heads - 1) / heads;
    int chunk = (d->cap + want - 1) / want;
    chunk = (chunk + kDecTile - 1) / kDecTile * kDecTile;
    if (chunk < kDecTile) chunk = kDecTile;
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

__device__ __forceinline__ void cp_async16_dec(void* smem, const void* gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

template <int G>
__global__ void __launch_bounds__(kDecThreads)
decode_split_kernel(const __nv_bfloat16* __restrict__ q, __nv_bfloat16* Kc, __nv_bfloat16* Vc,
                    const int32_t* __restrict__ len, const __nv_bfloat16* __restrict__ k_new,
                    const __nv_bfloat16* __restrict__ v_new, int H, int Hkv, int cap,
                    int64_t kv_sb, int64_t kv_sh, float scale_log2, int chunk, int nsplit,
                    float* __restrict__ ws_o, float* __restrict__ ws_ml, float* __restrict__ ws_s,
                    int want_logits, int32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem[];
    // layout: 2 stages x (K tile, V tile) of 64 padded rows, then q [G][128] f32, S [G][64] f32
    unsigned char* stage_base = smem;
    constexpr int kTileBytes = kDecTile * kRowPad;
    float* qs = reinterpret_cast<float*>(smem + 4 * kTileBytes);
    float* S = qs + G * kHeadDim;
    float* corr = S + G * kDecTile;                  // [0..8) rescale, [8..16) tile sums, [16..24) running max
    float* red = corr + 32;                          // [4 warps][G][128] final reduction

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
    for (int i = tid; i < G * kHeadDim; i += kDecThreads)
        qs[i] = __bfloat162float(q[(int64_t)(b * H + h0) * kHeadDim + i]) * scale_log2;

    const int ntile = (j_end - j_begin + kDecTile - 1) / kDecTile;
    auto issue_tile = [&](int t) {
        unsigned char* ks = stage_base + (t & 1) * 2 * kTileBytes;
        unsigned char* vs = ks + kTileBytes;
        const int j0 = j_begin + t * kDecTile;
        // 64 rows x 16 vectors per tensor; thread -> (row = i/16, vec = i%16)
        for (int i = tid; i < kDecTile * 16; i += kDecThreads) {
            const int rr = i >> 4, vv = i & 15;
            const int j = j0 + rr;
            if (j < j_end) {
                const __nv_bfloat16* ksrc = (append && j == ln) ? kn : Kseq + (int64_t)j * kHeadDim;
                const __nv_bfloat16* vsrc = (append && j == ln) ? vn : Vseq + (int64_t)j * kHeadDim;
                cp_async16_dec(ks + rr * kRowPad + vv * 16, ksrc + vv * 8);
                cp_async16_dec(vs + rr * kRowPad + vv * 16, vsrc + vv * 8);
            }
        }
        cp_async_commit();
    };
    issue_tile(0);
    if (ntile > 1) issue_tile(1);

    float m_run[G], l_run[G];                         // replicated per thread (same in all threads)
    float acc[G][4];
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
        m_run[hh] = -INFINITY; l_run[hh] = 0.f;
        acc[hh][0] = acc[hh][1] = acc[hh][2] = acc[hh][3] = 0.f;
    }

    for (int t = 0; t < ntile; ++t) {
        if (t + 1 < ntile) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncthreads();
        const unsigned char* ks = stage_base + (t & 1) * 2 * kTileBytes;
        const unsigned char* vs = ks + kTileBytes;
        const int j0 = j_begin + t * kDecTile;
        const int valid = min(kDecTile, j_end - j0);
        // ---- logits: thread -> key (tid & 63), heads hh = (tid >> 6), +2, ...
        {
            const int jj = tid & 63, half = tid >> 6;
            float s[(G + 1) / 2];
#pragma unroll
            for (int u = 0; u < (G + 1) / 2; ++u) s[u] = 0.f;
            if (jj < valid) {
                const uint4* krow = reinterpret_cast<const uint4*>(ks + jj * kRowPad);
#pragma unroll 4
                for (int v = 0; v < 16; ++v) {
                    const uint4 x = krow[v];
                    const float k0 = bf16_lo(x.x), k1 = bf16_hi(x.x), k2 = bf16_lo(x.y), k3 = bf16_hi(x.y);
                    const float k4 = bf16_lo(x.z), k5 = bf16_hi(x.z), k6 = bf16_lo(x.w), k7 = bf16_hi(x.w);
#pragma unroll
                    for (int u = 0; u < (G + 1) / 2; ++u) {
                        const int hh = half + 2 * u;
                        if (hh < G) {
                            const float4 qa = *reinterpret_cast<const float4*>(qs + hh * kHeadDim + v * 8);
                            const float4 qb = *reinterpret_cast<const float4*>(qs + hh * kHeadDim + v * 8 + 4);
                            s[u] = fmaf(k0, qa.x, s[u]); s[u] = fmaf(k1, qa.y, s[u]);
                            s[u] = fmaf(k2, qa.z, s[u]); s[u] = fmaf(k3, qa.w, s[u]);
                            s[u] = fmaf(k4, qb.x, s[u]); s[u] = fmaf(k5, qb.y, s[u]);
                            s[u] = fmaf(k6, qb.z, s[u]); s[u] = fmaf(k7, qb.w, s[u]);
                        }
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < (G + 1) / 2; ++u) {
                const int hh = half + 2 * u;
                if (hh < G) {
                    S[hh * kDecTile + jj] = jj < valid ? s[u] : -INFINITY;
                    if (want_logits && jj < valid)
                        ws_s[(int64_t)(b * H + h0 + hh) * cap + j0 + jj] = s[u];
                }
            }
        }
        __syncthreads();
        // ---- online softmax: warp w handles heads w, w+4
        for (int hh = warp; hh < G; hh += 4) {
            const float s0 = S[hh * kDecTile + lane], s1 = S[hh * kDecTile + lane + 32];
            float mx = fmaxf(s0, s1);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            const float m_old = (t == 0) ? -INFINITY : corr[16 + hh];
            const float m_new = fmaxf(m_old, mx);
            const float p0 = exp2f(s0 - m_new), p1 = exp2f(s1 - m_new);
            S[hh * kDecTile + lane] = p0; S[hh * kDecTile + lane + 32] = p1;
            float ps = p0 + p1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xFFFFFFFFu, ps, o);
            if (lane == 0) {
                corr[hh] = exp2f(m_old - m_new);          // 0 on the first tile
                corr[8 + hh] = ps;
                corr[16 + hh] = m_new;
            }
        }
        __syncthreads();
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
            const float c = corr[hh];
            l_run[hh] = l_run[hh] * c + corr[8 + hh];
            m_run[hh] = corr[16 + hh];
            acc[hh][0] *= c; acc[hh][1] *= c; acc[hh][2] *= c; acc[hh][3] *= c;
        }
        // ---- P x V: warp w takes keys w*16 .. w*16+15 of the tile, lane takes 4 dims
        {
            const int jb = warp * 16;
#pragma unroll 4
            for (int jj = jb; jj < jb + 16; ++jj) {
                if (jj < valid) {
                    const uint2 x = *reinterpret_cast<const uint2*>(vs + jj * kRowPad + lane * 8);
                    const float v0 = bf16_lo(x.x), v1 = bf16_hi(x.x), v2 = bf16_lo(x.y), v3 = bf16_hi(x.y);
#pragma unroll
                    for (int hh = 0; hh < G; ++hh) {
                        const float p = S[hh * kDecTile + jj];
                        acc[hh][0] = fmaf(p, v0, acc[hh][0]); acc[hh][1] = fmaf(p, v1, acc[hh][1]);
                        acc[hh][2] = fmaf(p, v2, acc[hh][2]); acc[hh][3] = fmaf(p, v3, acc[hh][3]);
                    }
                }
            }
        }
        __syncthreads();
        if (t + 2 < ntile) issue_tile(t + 2);
    }
    // ---- add the four warps' partial outputs in warp order, park the split's result
#pragma unroll
    for (int hh = 0; hh < G; ++hh)
        *reinterpret_cast<float4*>(red + ((warp * G + hh) * kHeadDim) + lane * 4) =
            make_float4(acc[hh][0], acc[hh][1], acc[hh][2], acc[hh][3]);
    __syncthreads();
    for (int i = tid; i < G * kHeadDim; i += kDecThreads) {
        const int hh = i / kHeadDim, dd = i % kHeadDim;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) v += red[(w * G + hh) * kHeadDim + dd];
        my_o[(int64_t)hh * nsplit * kHeadDim + dd] = v;
    }
    if (tid < G) {
        my_ml[(int64_t)tid * nsplit * 2] = m_run[tid];
        my_ml[(int64_t)tid * nsplit * 2 + 1] = l_run[tid];
    }
}

template <int G>
__global__ void __launch_bounds__(kDecThreads)
decode_combine_kernel(int32_t* len, int has_append, float* acc_score, int H, int Hkv, int cap,
                      int nsplit, const float* __restrict__ ws_o, const float* __restrict__ ws_ml,
                      const float* __restrict__ ws_s, __nv_bfloat16* __restrict__ out) {
    __shared__ float sM[G], sInvL[G];
    const int g = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int hd = b * Hkv + g;
    int ln = len[hd];
    if (ln < 0 || ln > cap) ln = 0;
    const bool append = has_append && ln < cap;
    const int ln_eff = ln + (append ? 1 : 0);
    const int h0 = g * G;
    if (tid < G) {
        const float* ml = ws_ml + (int64_t)(b * H + h0 + tid) * nsplit * 2;
        float M = -INFINITY;
        for (int s = 0; s < nsplit; ++s) M = fmaxf(M, ml[2 * s]);
        float Lsum = 0.f;
        for (int s = 0; s < nsplit; ++s)
            if (ml[2 * s + 1] > 0.f) Lsum += ml[2 * s + 1] * exp2f(ml[2 * s] - M);
        sM[tid] = M;
        sInvL[tid] = Lsum > 0.f ? 1.0f / Lsum : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
        const float* ml = ws_ml + (int64_t)(b * H + h0 + hh) * nsplit * 2;
        const float* po = ws_o + (int64_t)(b * H + h0 + hh) * nsplit * kHeadDim;
        float v = 0.f;
        for (int s = 0; s < nsplit; ++s)
            if (ml[2 * s + 1] > 0.f) v += po[s * kHeadDim + tid] * exp2f(ml[2 * s] - sM[hh]);
        out[(int64_t)(b * H + h0 + hh) * kHeadDim + tid] = __float2bfloat16_rn(v * sInvL[hh]);
    }
    if (acc_score) {
        float* acc = acc_score + (int64_t)hd * cap;
        for (int j = tid; j < ln_eff; j += kDecThreads) {
            float p = 0.f;
#pragma unroll
            for (int hh = 0; hh < G; ++hh)
                p += exp2f(ws_s[(int64_t)(b * H + h0 + hh) * cap + j] - sM[hh]) * sInvL[hh];
            const float old = (append && j == ln) ? 0.f : acc[j];     // a new entry starts at zero
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
    const size_t smem = 4 * (size_t)kDecTile * kRowPad + (size_t)G * kHeadDim * 4 +
                        (size_t)G * kDecTile * 4 + 32 * 4 + 4 * (size_t)G * kHeadDim * 4;
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(decode_split_kernel<G>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_split_kernel<G><<<dim3(L.nsplit, d->Hkv, d->B), kDecThreads, smem, stream>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(Kc),
        static_cast<__nv_bfloat16*>(Vc), len, static_cast<const __nv_bfloat16*>(k_new),
        static_cast<const __nv_bfloat16*>(v_new), d->H, d->Hkv, d->cap, kv_sb, kv_sh,
        scale * kLog2e, L.chunk, L.nsplit, ws_o, ws_ml, ws_s, acc_score != nullptr, dev_status);
    if (cudaGetLastError() != cudaSuccess) return LVLM_ERR_CUDA;
    decode_combine_kernel<G><<<dim3(d->Hkv, d->B), kDecThreads, 0, stream>>>(
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
