// In-place row compaction shared by lvlm_merge_compact (hidden states, K, V) and
// lvlm_kv_compress (K, V).
#pragma once
#include "common.cuh"

namespace lvlm {

// Compacts B*G (*2 when base1 != NULL) sequences of rows in place.  Sequence (b, g) of tensor
// t lives at base_t + b*stride_b + g*stride_g (bytes), rows of V 16-byte vectors.
// Output row o of a sequence takes input row src_map[m][o] (m = b when maps_per_g == 1, else
// b*G+g; map rows are map_stride ints apart); src < 0 marks the merged row, which receives
// sum_j wgt[b][j] * row(i0+j) over the n image tokens (wgt == NULL: no merged row).  With wgt the
// walk needs dst_map[b][i] as well: the output row of input row i, -1 for a merged row.
// meta[m*meta_stride] = first row whose content changes.  nout == NULL: every sequence has
// `Nout` rows after the call, else nout[m].  N = valid rows before the call.
lvlm_status launch_inplace_compact(void* base0, void* base1, int64_t stride_b, int64_t stride_g,
                                   int B, int G, int V, int Nout, const int32_t* src_map,
                                   const float* wgt, const int32_t* meta, int N, int n, int i0,
                                   int merged_row, int meta_stride, cudaStream_t stream,
                                   int maps_per_g = 1, int64_t map_stride = -1,
                                   const int32_t* nout = nullptr, const int32_t* dst_map = nullptr);

}  // namespace lvlm
