// Pieces of lvlm_merge_compact shared between its merge modes.
#pragma once
#include "common.cuh"

namespace lvlm {

constexpr int kMetaInts = 4;           // per sequence: first moved row, ticket counter, merged token, spare

// Launch shape of the kernel that streams the hidden states by input row.
struct HiddenGrid { int V, cps, cl, rpc; };   // 16-byte groups per row, CTAs per sequence, cluster size, rows per CTA
HiddenGrid hidden_grid(const lvlm_dims* d);

// Reads every input row of `hidden` once.  dst_map[b][i] >= 0: the row is copied to that row of
// hidden_out; == -1: it is added, times wgt, to the merged row P_new at row i0+k (wgt != NULL);
// <= -2: it is copied to row -dst-2 of `scratch` (scratch != NULL).  Strides in elements.
lvlm_status launch_hidden_rows(const void* hidden, void* hidden_out, int64_t hid_sb, int64_t out_sb,
                               const lvlm_dims* d, const HiddenGrid& L, const int32_t* dst_map,
                               const float* wgt, int32_t* meta, float* partial, void* scratch,
                               int64_t scr_sb, cudaStream_t stream);

// lvlm_merge_compact in mode LVLM_W_NEAREST_KEPT (nearest_kept.cu).
size_t nearest_kept_workspace(const lvlm_dims* d);
lvlm_status launch_nearest_kept(const void* hidden, void* hidden_out, void* Kc, void* Vc, int32_t* pos_ids,
                                const int32_t* rank, const lvlm_dims* d, float* mass, int32_t* new_len,
                                void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t stream);

}  // namespace lvlm
