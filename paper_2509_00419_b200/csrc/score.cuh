// Declarations shared by the scoring kernels.
#pragma once
#include "common.cuh"

namespace lvlm {

struct ScoreLayout { size_t off_partial, off_lse, total; };
struct ScoreStrides { int64_t q_sb, q_sn, q_sh, kv_sb, kv_sh; };   // elements

bool score_layout(const lvlm_dims* d, ScoreLayout* L);

lvlm_status launch_score_reduce(const float* partial, const lvlm_dims* d, float* score,
                                float* score_head, int32_t* dev_status, cudaStream_t stream);

}  // namespace lvlm
