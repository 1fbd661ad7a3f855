// In-place row compaction shared by lvlm_merge_compact (hidden states, K, V) and
// lvlm_kv_compress (K, V).
#pragma once
#include "common.cuh"

namespace lvlm {

// Compacts B*G (*2 when base1 != NULL) sequences of rows in place.  Sequence (b, g) of tensor t
// lives at base_t + b*stride_b + g*stride_g (bytes), rows of V 16-byte vectors, packed.
struct CompactJob {
    void* base0 = nullptr;
    void* base1 = nullptr;
    int64_t stride_b = 0, stride_g = 0;
    int B = 0, G = 1, V = 0;
    // Output row o of a sequence takes input row src_map[m][o] (>= o), m = b when maps_per_g == 1, else
    // b*G+g; map rows are map_stride ints apart.  src < 0 marks the merged row (see `partial`).
    const int32_t* src_map = nullptr;
    int maps_per_g = 1;
    int64_t map_stride = 0;
    const int32_t* meta = nullptr;      // meta[m*meta_stride] = first row whose content changes
    int meta_stride = 1;
    const int32_t* nout = nullptr;      // rows after the call per map, or NULL: Nout for every sequence
    int Nout = 0;
    int N = 0;                          // upper bound of the rows of a sequence (sizes the launch)
    // The merged row, if any: row `merged_row` of every sequence receives the sum, rounded once to bf16, of
    // the P fp32 partial rows partial[(((b*G+g)*T+t)*P + p)*V*8 ...], p = 0..P-1 in that order (T = tensors).
    int merged_row = -1;
    const float* partial = nullptr;
    int P = 0;
    // Optionally up to two arrays of 4-byte words per sequence map (maps_per_g != 1), rows map_stride words apart:
    // words [meta, nout) of side_src[i] are copied to side_dst[i] (compacted out of place by the kernel before).
    void* side_dst[2] = {nullptr, nullptr};
    const void* side_src[2] = {nullptr, nullptr};
    // Optionally, in the same launch: row `fin_row` of every sequence of another tensor (rows of fin_V 16-byte
    // vectors, sequences fin_stride_b bytes apart) receives the sum of the fin_P partial rows
    // fin_partial[(b*fin_P + p)*fin_V*8 ...].  base0 may be NULL then: nothing is compacted.
    // The maps, meta and nout were complete, and the rows were no longer written, before the kernel ahead of this
    // launch in the stream let it start (that kernel only reads the rows): the first rows are then fetched while it
    // still runs; the partial rows and every write wait for it.
    bool maps_ready = false;
    void* fin_base = nullptr;
    int64_t fin_stride_b = 0;
    int fin_row = 0, fin_V = 0, fin_P = 0;
    const float* fin_partial = nullptr;
};

lvlm_status launch_inplace_compact(const CompactJob& job, cudaStream_t stream);

}  // namespace lvlm
