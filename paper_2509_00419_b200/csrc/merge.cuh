// Pieces of lvlm_merge_compact shared between its merge modes.
#pragma once
#include "common.cuh"

namespace lvlm {

constexpr int kMetaInts = 4;           // per sequence: first moved row, ticket counter, merged token, spare

// Launch shape of the kernel that streams the hidden states by input row: 16-byte groups per row, CTAs per
// sequence, cluster size, rows per tile, bytes of a tile's slot in shared memory, tiles in flight.
struct HiddenGrid { int V, cps, cl, rpt, slotB, nstage; };
HiddenGrid hidden_grid(const lvlm_dims* d);

// This layer's K and V for the same launch: the rows merged away are added, times wgt, per (sequence, KV
// head, K|V) into kvP fp32 partial rows (chunks of the image span), kv_partial[b][g][K|V][chunk][128].
struct StreamKv { const void* K; const void* V; int64_t kv_sb, kv_sh; int Hkv, kvP; float* kv_partial; };

// Reads every input row of `hidden` once.  dst_map[b][i] >= 0: the row is copied to that row of
// hidden_out; == -1: it is added, times wgt, to the merged row P_new at row i0+k (wgt != NULL);
// <= -2: it is copied to row -dst-2 of `scratch` (scratch != NULL).  Strides in elements.
// hidden_out == NULL: nothing is stored, only the merged rows are read and one fp32 partial row per cluster
// is left in `partial` ([B][*partials_out][C]) for the in-place compaction that follows.  L gives the launch
// shape at most: fewer CTAs are used when the device cannot run that many clusters at a time.
lvlm_status launch_hidden_rows(const void* hidden, void* hidden_out, int64_t hid_sb, int64_t out_sb,
                               const lvlm_dims* d, const HiddenGrid& L, const int32_t* dst_map,
                               const float* wgt, int32_t* meta, float* partial, void* scratch,
                               int64_t scr_sb, cudaStream_t stream, const StreamKv* kv = nullptr,
                               int32_t* dev_status = nullptr, int* partials_out = nullptr);

// lvlm_merge_compact in mode LVLM_W_NEAREST_KEPT (nearest_kept.cu).
size_t nearest_kept_workspace(const lvlm_dims* d);
lvlm_status launch_nearest_kept(const void* hidden, void* hidden_out, void* Kc, void* Vc, int32_t* pos_ids,
                                const int32_t* rank, const lvlm_dims* d, float* mass, int32_t* new_len,
                                void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t stream);

}  // namespace lvlm
