// lvlm_score_tokens: attention mass each image key receives from a window of query rows,
// averaged over heads (Section 3.2.1, paragraph 3).
//
// Argument checks, workspace layout and the entry point; the kernels are in score_tc.cu.
#include "common.cuh"
#include "score.cuh"

namespace lvlm {

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

}  // namespace lvlm

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
    float* lse_ws = reinterpret_cast<float*>(wsb + L.off_lse);
    return launch_score_tc(Q, K, lse, d, st, scale, lse_ws, partial,
                           reinterpret_cast<int32_t*>(wsb + L.off_cnt), score, score_head, dev_status, stream);
}
