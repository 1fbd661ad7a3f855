// lvlm_score_tokens: attention mass each image key receives from a window of query rows,
// averaged over heads (Section 3.2.1, paragraph 3).
//
// Two launches: a per-(sequence, head) kernel produces the column sums of that head's
// attention probabilities over the image span; a reduction kernel averages over heads
// (score) and sums over each KV group (score_head), in a fixed order.
#include "common.cuh"
#include "score.cuh"

namespace lvlm {

constexpr float kLog2eS = 1.4426950408889634f;
constexpr int kRefRows = 128;       // query rows per pass of the CUDA-core kernel (one per thread)
constexpr int kRefKeys = 32;        // keys staged per tile

bool score_layout(const lvlm_dims* d, ScoreLayout* L) {
    if (!d || d->B <= 0 || d->H <= 0 || d->Hkv <= 0 || d->H % d->Hkv || d->N <= 0 || d->n <= 0 ||
        d->i0 < 0 || (int64_t)d->i0 + d->n > d->N || d->q_lo < 0 || d->q_lo >= d->q_hi ||
        d->q_hi > d->N || d->cap < d->N)
        return false;
    size_t off = 0;
    L->off_partial = off; off = align_up(off + (size_t)d->B * d->H * d->n * 4, 256);
    L->off_lse = off;     off = align_up(off + (size_t)d->B * d->H * (d->q_hi - d->q_lo) * 4, 256);
    L->off_cnt = off;     off = align_up(off + (size_t)d->B * ((d->n + 127) / 128) * 4, 256);
    L->total = off;
    return true;
}

size_t score_tokens_workspace(const lvlm_dims* d) {
    ScoreLayout L;
    return score_layout(d, &L) ? L.total : 0;
}

// CUDA-core scoring kernel: grid (H, B), 128 threads, thread = one query row of the current
// block of 128 rows.  Pass 1 finds each row's softmax normaliser over the keys it sees, pass 2
// adds exp(logit - normaliser) of every image key over the rows.  Slow and simple: it is the
// cross-check of the tensor-core kernel and serves shapes that kernel does not take.
__global__ void __launch_bounds__(kRefRows)
score_colsum_simt_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                         const float* __restrict__ lse, int H, int G, int N, int i0, int n,
                         int q_lo, int q_hi, int causal, int64_t q_sb, int64_t q_sn, int64_t q_sh,
                         int64_t kv_sb, int64_t kv_sh, float scale_log2, float* __restrict__ partial) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* colsum = reinterpret_cast<float*>(smem_raw);                 // [n]
    uint4* ktile = reinterpret_cast<uint4*>(colsum + ((n + 3) & ~3));   // [32 keys][16 vectors]
    float* wsum = reinterpret_cast<float*>(ktile + kRefKeys * 16);      // [4 warps][32 keys]

    pdl_enter();
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int Nq = q_hi - q_lo;
    const __nv_bfloat16* Kseq = K + (int64_t)b * kv_sb + (int64_t)(h / G) * kv_sh;
    for (int j = tid; j < n; j += kRefRows) colsum[j] = 0.f;

    for (int r0 = 0; r0 < Nq; r0 += kRefRows) {
        const int i = r0 + tid;
        const bool row_ok = i < Nq;
        const int pos = q_lo + (row_ok ? i : Nq - 1);
        float qf[kHeadDim];
        {
            const uint4* qrow = reinterpret_cast<const uint4*>(
                Q + (int64_t)b * q_sb + (int64_t)(row_ok ? i : Nq - 1) * q_sn + (int64_t)h * q_sh);
#pragma unroll
            for (int v = 0; v < 16; ++v) {
                const uint4 x = qrow[v];
                qf[v * 8 + 0] = bf16_lo(x.x) * scale_log2; qf[v * 8 + 1] = bf16_hi(x.x) * scale_log2;
                qf[v * 8 + 2] = bf16_lo(x.y) * scale_log2; qf[v * 8 + 3] = bf16_hi(x.y) * scale_log2;
                qf[v * 8 + 4] = bf16_lo(x.z) * scale_log2; qf[v * 8 + 5] = bf16_hi(x.z) * scale_log2;
                qf[v * 8 + 6] = bf16_lo(x.w) * scale_log2; qf[v * 8 + 7] = bf16_hi(x.w) * scale_log2;
            }
        }
        const int last_pos = q_lo + min(Nq, r0 + kRefRows) - 1;
        const int key_end = causal ? min(N, last_pos + 1) : N;
        const int my_end = causal ? pos + 1 : N;             // keys [0, my_end) are visible

        auto load_tile = [&](int j0) {
            __syncthreads();
            for (int e = tid; e < kRefKeys * 16; e += kRefRows) {
                const int jj = e >> 4, v = e & 15;
                const int j = j0 + jj;
                ktile[e] = j < N ? reinterpret_cast<const uint4*>(Kseq + (int64_t)j * kHeadDim)[v]
                                 : make_uint4(0, 0, 0, 0);
            }
            __syncthreads();
        };
        auto dot = [&](int jj) {                              // logit of staged key jj (log2 domain)
            float a = 0.f;
#pragma unroll
            for (int v = 0; v < 16; ++v) {
                const uint4 x = ktile[jj * 16 + v];
                a = fmaf(qf[v * 8 + 0], bf16_lo(x.x), a); a = fmaf(qf[v * 8 + 1], bf16_hi(x.x), a);
                a = fmaf(qf[v * 8 + 2], bf16_lo(x.y), a); a = fmaf(qf[v * 8 + 3], bf16_hi(x.y), a);
                a = fmaf(qf[v * 8 + 4], bf16_lo(x.z), a); a = fmaf(qf[v * 8 + 5], bf16_hi(x.z), a);
                a = fmaf(qf[v * 8 + 6], bf16_lo(x.w), a); a = fmaf(qf[v * 8 + 7], bf16_hi(x.w), a);
            }
            return a;
        };

        float m = -INFINITY, l = 0.f;
        if (lse) {
            m = lse[((int64_t)b * H + h) * Nq + (row_ok ? i : Nq - 1)] * kLog2eS;
            l = 1.f;
        } else {
            for (int j0 = 0; j0 < key_end; j0 += kRefKeys) {
                load_tile(j0);
#pragma unroll 1
                for (int jj = 0; jj < kRefKeys; ++jj) {
                    if (j0 + jj < my_end) {
                        const float sv = dot(jj);
                        const float m_new = fmaxf(m, sv);
                        l = l * exp2f(m - m_new) + exp2f(sv - m_new);
                        m = m_new;
                    }
                }
            }
        }
        const float inv_l = (row_ok && l > 0.f) ? 1.0f / l : 0.f;
        const int img_end = min(i0 + n, key_end);
        for (int j0 = i0; j0 < img_end; j0 += kRefKeys) {
            load_tile(j0);
#pragma unroll 1
            for (int jj = 0; jj < kRefKeys; ++jj) {
                float p = 0.f;
                if (j0 + jj < my_end && j0 + jj < img_end) p = exp2f(dot(jj) - m) * inv_l;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xFFFFFFFFu, p, o);
                if (lane == 0) wsum[warp * kRefKeys + jj] = p;
            }
            __syncthreads();
            if (tid < kRefKeys && j0 + tid < img_end)
                colsum[j0 - i0 + tid] += (wsum[tid] + wsum[kRefKeys + tid]) +
                                         (wsum[2 * kRefKeys + tid] + wsum[3 * kRefKeys + tid]);
        }
        __syncthreads();
    }
    __syncthreads();
    float* dst = partial + ((int64_t)b * H + h) * n;
    for (int j = tid; j < n; j += kRefRows) dst[j] = colsum[j];
}

// partial holds P rows per sequence, G consecutive rows per KV group (P = H, G = group size for
// per-head partials; P = Hkv, G = 1 for group-summed partials).
// score[b,j] = inv_h * sum_p partial[b,p,j];  score_head[b,g,j] = sum_{p in g} partial[b,p,j].
__global__ void score_reduce_kernel(const float* __restrict__ partial, int P, int G, int n,
                                    float inv_h, float* __restrict__ score,
                                    float* __restrict__ score_head, int64_t head_stride,
                                    int32_t* dev_status) {
    pdl_enter();
    const int b = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const int Hkv = P / G;
    float tot = 0.f;
    for (int g = 0; g < Hkv; ++g) {
        float gs = 0.f;
        for (int hh = 0; hh < G; ++hh) gs += partial[((int64_t)b * P + g * G + hh) * n + j];
        if (score_head) score_head[((int64_t)b * Hkv + g) * head_stride + j] = gs;
        tot += gs;
    }
    const float s = tot * inv_h;
    score[(int64_t)b * n + j] = s;
    if (dev_status && (__float_as_uint(s) & 0x7F800000u) == 0x7F800000u)
        atomicOr(dev_status, LVLM_DEV_NONFINITE);
}

lvlm_status launch_score_simt(const void* Q, const void* K, const float* lse, const lvlm_dims* d,
                              const ScoreStrides& st, float scale, float* partial,
                              cudaStream_t stream) {
    const size_t smem = (size_t)((d->n + 3) & ~3) * 4 + kRefKeys * 16 * 16 + 4 * kRefKeys * 4;
    if (smem > (size_t)kMaxDynSmem) return LVLM_ERR_UNSUPPORTED;
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(score_colsum_simt_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    return launch_kernel(score_colsum_simt_kernel, dim3(d->H, d->B), dim3(kRefRows), smem, stream, 1,
                         static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K), lse, d->H,
                         d->H / d->Hkv, d->N, d->i0, d->n, d->q_lo, d->q_hi, d->causal, st.q_sb, st.q_sn, st.q_sh,
                         st.kv_sb, st.kv_sh, scale * kLog2eS, partial);
}

lvlm_status launch_score_reduce(const float* partial, bool group_summed, const lvlm_dims* d,
                                float* score, float* score_head, int32_t* dev_status,
                                cudaStream_t stream) {
    return launch_kernel(score_reduce_kernel, dim3((d->n + 255) / 256, d->B), dim3(256), 0, stream, 1,
                         partial, group_summed ? d->Hkv : d->H, group_summed ? 1 : d->H / d->Hkv, d->n,
                         1.0f / (float)d->H, score, score_head,
                         d->head_stride ? d->head_stride : (int64_t)d->n, dev_status);
}

}  // namespace lvlm

// Selects the scoring kernel: 1 = CUDA-core cross-check kernel, anything else = the tensor-core
// kernel (the product path).  Test hook; not part of the public header.
static int g_score_impl = 0;
extern "C" void lvlm_debug_set_score_impl(int impl) { g_score_impl = impl; }

extern "C" lvlm_status lvlm_score_tokens(const void* Q, const void* K, const float* lse,
                                          const lvlm_dims* d, float scale, float* score,
                                          float* score_head, void* ws, size_t ws_bytes,
                                          int32_t* dev_status, void* stream_) {
    using namespace lvlm;
    cudaStream_t stream = (cudaStream_t)stream_;
    ScoreLayout L;
    if (!Q || !K || !score || !score_layout(d, &L)) return LVLM_ERR_INVALID_ARG;
    if (d->D != kHeadDim) return LVLM_ERR_UNSUPPORTED;
    if (d->head_stride != 0 && d->head_stride < d->n) return LVLM_ERR_INVALID_ARG;
    ScoreStrides st;
    const int Nq = d->q_hi - d->q_lo;
    st.q_sh = d->q_stride_h ? d->q_stride_h : d->D;
    st.q_sn = d->q_stride_n ? d->q_stride_n : (int64_t)d->H * d->D;
    st.q_sb = d->q_stride_b ? d->q_stride_b : (int64_t)Nq * st.q_sn;
    st.kv_sh = d->kv_stride_h ? d->kv_stride_h : (int64_t)d->cap * d->D;
    st.kv_sb = d->kv_stride_b ? d->kv_stride_b : (int64_t)d->Hkv * st.kv_sh;
    if (!aligned16(Q) || !aligned16(K) || st.q_sh % 8 || st.q_sn % 8 || st.q_sb % 8 ||
        st.kv_sh % 8 || st.kv_sb % 8)
        return LVLM_ERR_ALIGNMENT;
    if (!ws || !aligned256(ws) || ws_bytes < L.total) return LVLM_ERR_WORKSPACE;
    char* wsb = static_cast<char*>(ws);
    float* partial = reinterpret_cast<float*>(wsb + L.off_partial);
    if (g_score_impl == 1) {
        lvlm_status s = launch_score_simt(Q, K, lse, d, st, scale, partial, stream);
        if (s != LVLM_OK) return s;
        return launch_score_reduce(partial, false, d, score, score_head, dev_status, stream);
    }
    float* lse_ws = reinterpret_cast<float*>(wsb + L.off_lse);
    return launch_score_tc(Q, K, lse, d, st, scale, lse_ws, partial,
                           reinterpret_cast<int32_t*>(wsb + L.off_cnt), score, score_head, dev_status, stream);
}
