// Declarations shared by the scoring kernels.
#pragma once
#include "common.cuh"

namespace lvlm {

struct ScoreLayout { size_t off_partial, off_lse, off_cnt, total; };
struct ScoreStrides { int64_t q_sb, q_sn, q_sh, kv_sb, kv_sh; };   // elements

bool score_layout(const lvlm_dims* d, ScoreLayout* L);

// Tensor-core path: pass 1 (row normalisers into lse_ws, skipped when the caller supplies lse) and
// pass 2 (column sums per CTA row into partial, added over the heads by the last CTA of each key
// tile, which writes score and score_head).  cnt holds one counter per (sequence, key tile).
// normalisers_ready: lse_ws already holds the log2-domain normalisers of the window rows (the attention kernel
// of lvlm_prefill_attn wrote them): pass 1 is skipped.
lvlm_status launch_score_tc(const void* Q, const void* K, const float* lse, const lvlm_dims* d,
                            const ScoreStrides& st, float scale, float* lse_ws, float* partial,
                            int32_t* cnt, float* score, float* score_head, int32_t* dev_status,
                            cudaStream_t stream, bool normalisers_ready = false);

}  // namespace lvlm
