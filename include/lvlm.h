/*
 * lvlm.h - C ABI of the LightVLM token-reduction / KV-cache-compression kernels (sm_100a).
 *
 * The library implements the computation that LightVLM adds to a vision-language model:
 * pyramid token merging during encoding (paper Section 3.2.1) and KV-cache compression
 * followed by decoding over the shortened cache (Section 3.2.2), with the settings of
 * Appendix A.2.  It does not contain a model: callers hand in the tensors of one layer.
 *
 * Conventions for every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library never
 *     allocates, frees or keeps a pointer after the call returns.  `lvlm_dims` itself is a
 *     HOST struct, read during the call only.
 *   - Scratch memory comes from the caller: `ws` (device, 256-byte aligned) of at least
 *     `lvlm_workspace_bytes(op, dims)` bytes.  Its contents need not be preserved or zeroed.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy
 *     default stream) and the call returns without synchronising.  Calls that share `ws` or
 *     any in/out tensor must be ordered by the caller (same stream is enough).
 *   - Activations are bf16, scores fp32, indices int32.  The innermost dimension of every
 *     tensor is contiguous and 16-byte aligned.  Only D == 128 is supported.
 *   - A host-detectable error returns a non-zero `lvlm_status` and enqueues nothing.
 *     Conditions only the device can see (non-finite score, length beyond capacity) OR a
 *     `LVLM_DEV_*` bit into `*dev_status` (optional, caller-owned int32 on the device,
 *     never cleared by the library); the offending access is skipped and the kernel ends
 *     normally.  No kernel traps or asserts.
 *   - Results are bit-reproducible from run to run: no floating-point atomics are used.
 */
#ifndef LVLM_H_
#define LVLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LVLM_OK = 0,
    LVLM_ERR_INVALID_ARG = 1,   /* NULL required pointer, size or range out of bounds */
    LVLM_ERR_UNSUPPORTED = 2,   /* D != 128, n or cache length beyond the built limits */
    LVLM_ERR_ALIGNMENT = 3,     /* pointer or stride not 16-byte aligned */
    LVLM_ERR_WORKSPACE = 4,     /* ws NULL, misaligned or smaller than lvlm_workspace_bytes */
    LVLM_ERR_CUDA = 5           /* a CUDA runtime call failed (launch, attribute, driver entry) */
} lvlm_status;

/* bits OR-ed into *dev_status by kernels */
enum { LVLM_DEV_NONFINITE = 1, LVLM_DEV_TIMEOUT = 2, LVLM_DEV_BOUNDS = 4 };

/* How the r+1 least important image tokens become one token (Section 3.2.1, paragraph 4).
 * p = 0 is the most important merged token; weights are divided by their sum.
 *   LINEAR_RANK   the stated weight list W_v = {r+1, r, ..., 1}                 (default)
 *   GEOMETRIC     (1/2, 1/4, ..., 2^-r, 2^-r): the literal result of repeatedly merging the
 *                 last two tokens of the queue with equal weights
 *   UNIFORM       1/(r+1) each
 *   CUSTOM        caller-supplied list w_custom[0..r]
 *   NEAREST_KEPT  not in the paper: each dropped token is averaged into the kept token with
 *                 the highest cosine similarity of the hidden rows (lower index wins ties),
 *                 weighted by the token masses; that layer's K and V rows are averaged with
 *                 the same assignment; no extra token.  Needs hidden_out (out of place),
 *                 1 <= k, n - k <= 65536, and a workspace sized with d->merge_mode set to it.
 *                 After the call the first B*(n-k) int32 of `ws` hold the assignment: for the
 *                 dropped tokens in ascending order, the index of their kept token in the
 *                 ascending list of kept tokens. */
typedef enum {
    LVLM_W_LINEAR_RANK = 0, LVLM_W_GEOMETRIC = 1, LVLM_W_UNIFORM = 2,
    LVLM_W_CUSTOM = 3, LVLM_W_NEAREST_KEPT = 4
} lvlm_merge_mode;

typedef enum {
    LVLM_OP_SCORE_TOKENS = 0, LVLM_OP_SELECT_TOPK = 1, LVLM_OP_MERGE_COMPACT = 2,
    LVLM_OP_KV_COMPRESS = 3, LVLM_OP_DECODE_ATTN = 4, LVLM_OP_PREFILL_ATTN = 5
} lvlm_op;

/* Problem sizes.  Each entry point lists the fields it reads; the others are ignored.
 * Strides are in ELEMENTS; 0 selects the packed default given beside the tensor. */
typedef struct lvlm_dims {
    int32_t B;        /* sequences in the batch */
    int32_t H;        /* query heads */
    int32_t Hkv;      /* key/value heads; H % Hkv == 0; query head h uses KV head h / (H/Hkv) */
    int32_t D;        /* head dimension (128) */
    int32_t N;        /* tokens per sequence before the call */
    int32_t C;        /* hidden channels, a multiple of 8 */
    int32_t cap;      /* rows allocated per (sequence, KV head) in a K or V cache */
    int32_t i0;       /* index of the first image token */
    int32_t n;        /* number of image tokens: the span is [i0, i0+n) */
    int32_t k;        /* image tokens kept intact (P_unmerged); the other n-k are merged */
    int32_t q_lo;     /* scoring: first query row (sequence position) of the window */
    int32_t q_hi;     /* scoring: one past the last query row of the window */
    int32_t causal;   /* scoring: 1 = row at position p sees keys j <= p; 0 = sees all N keys */
    int32_t recent;   /* kv_compress: this many newest entries of every head are never evicted */
    int32_t merge_mode; /* lvlm_workspace_bytes(LVLM_OP_MERGE_COMPACT): the lvlm_merge_mode to size for */
    int32_t cache_stable; /* decode_attn: 1 = Kc, Vc and len are neither written nor still being read by the
                             operation enqueued just before this call (see lvlm_decode_attn) */
    int64_t q_stride_b, q_stride_n, q_stride_h;  /* Q[b][i][h][D]; default packed [B][q_hi-q_lo][H][D] */
    int64_t kv_stride_b, kv_stride_h;            /* K,V[b][g][row][D], rows packed; default [B][Hkv][cap][D] */
    int64_t hid_stride_b;                        /* hidden[b][row][C], rows packed; default N*C */
    int64_t out_stride_b;                        /* hidden_out[b][row][C]; default (rows after the call)*C */
    int64_t head_stride;                         /* score_head[b][g] rows; default n */
} lvlm_dims;

/* Library version string (static storage). */
const char* lvlm_version(void);

/* Text for a status code (static storage). */
const char* lvlm_status_string(lvlm_status s);

/* Bytes of device scratch `op` needs for `d` (0 if `d` is invalid for that op).  Host only. */
size_t lvlm_workspace_bytes(int op, const lvlm_dims* d);

/*
 * Importance of every image token: the attention it receives, summed over the query rows
 * of a window and averaged over heads (Section 3.2.1, paragraph 3: the per-key "cumsum
 * attention scores" A, "averaged ... across different heads").
 *
 *   s_head[b,h,j] = sum_{p in [q_lo,q_hi)} softmax_over_visible_keys(q[b,p,h] . K[b,h/G] * scale)[j]
 *   score[b,j-i0]          = (1/H) sum_h s_head[b,h,j]                     j in [i0, i0+n)
 *   score_head[b,g,j-i0]   = sum_{h in group g} s_head[b,h,j]   (what per-head KV compression uses)
 *
 * The softmax of row p is taken over ALL keys it can see (j <= p if d->causal, else all N),
 * not only over image keys.  The window [0,N) gives the column sums of the full causal
 * attention matrix; the window [i0+n, N) gives the attention of the instruction text only.
 *   Q          [B][q_hi-q_lo][H][D] bf16, row 0 = sequence position q_lo (strides d->q_stride_*)
 *   K          [B][Hkv][cap][D] bf16, rows 0..N-1 valid (strides d->kv_stride_*)
 *   lse        optional [B][H][q_hi-q_lo] fp32: natural-log sum-exp of each row's scaled
 *              logits as produced by the attention kernel that ran before; NULL = computed here
 *   score      [B][n] fp32 out;  score_head optional [B][Hkv] rows of n fp32 out, d->head_stride apart
 *              (a caller can point it at acc_score + i0 of a cache with head_stride = cap)
 * Reads d: B,H,Hkv,D,N,cap,i0,n,q_lo,q_hi,causal,q_stride_*,kv_stride_*,head_stride.
 * Errors: INVALID_ARG (NULL Q/K/score, i0+n>N, q_lo>=q_hi, q_hi>N, N>cap, H%Hkv), UNSUPPORTED
 * (D!=128), ALIGNMENT, WORKSPACE.  A non-finite score sets LVLM_DEV_NONFINITE.
 */
lvlm_status lvlm_score_tokens(const void* Q, const void* K, const float* lse,
                              const lvlm_dims* d, float scale,
                              float* score, float* score_head,
                              void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * The attention of a prefill layer with the importance scores as its by-product (Section 3.2.1, paragraph 3 and
 * its footnote: the per-key summed scores are what the attention kernel of the layer returns anyway, "to avoid
 * incurring additional massive computations").  Computes, for every sequence position p and query head h,
 *     out[b,p,h,:] = softmax_over_visible_keys(Q[b,p,h] . K[b,h/G] * scale) V[b,h/G]
 *     lse[b,h,p]   = natural log of the sum of the exponentials of row p's scaled logits
 * and, when `score` is given, exactly what lvlm_score_tokens computes for the window [q_lo, q_hi) of the same
 * rows - but from the normalisers this attention pass has just produced, so that only the column-sum pass
 * over the window is paid on top of the attention.
 *   Q          [B][N][H][D] bf16, row p = sequence position p (strides d->q_stride_*)
 *   K, V       [B][Hkv][cap][D] bf16, rows 0..N-1 valid (strides d->kv_stride_*)
 *   out        [B][N][H][D] bf16, packed        lse  [B][H][N] fp32
 *   score      optional [B][n] fp32; score_head optional [B][Hkv] rows of n fp32, d->head_stride apart
 *              (needs score); the workspace is only needed with score
 * Reads d: B,H,Hkv,D,N,cap,causal,q_stride_*,kv_stride_*, and with score also i0,n,q_lo,q_hi,head_stride.
 * Errors: INVALID_ARG (NULL Q/K/V/out/lse, N>cap, H%Hkv, scale<=0, score_head without score, a bad window),
 * UNSUPPORTED (D!=128), ALIGNMENT, WORKSPACE.  Contents of the outputs are undefined when a kernel gave up
 * on a wait and set LVLM_DEV_TIMEOUT (the same holds for lvlm_score_tokens and lvlm_merge_compact).
 */
lvlm_status lvlm_prefill_attn(const void* Q, const void* K, const void* V, const lvlm_dims* d, float scale,
                              void* out, float* lse, float* score, float* score_head,
                              void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Split of the image tokens into P_unmerged and P_merged (Section 3.2.1, paragraph 4): the
 * total order of the n tokens by (score descending, index ascending).
 *   score     [B] rows of n fp32, row stride score_stride elements (0 = n)
 *   rank      [B][n] int32 out: position of token j in the order.  rank < k: kept intact;
 *             rank >= k: merged, and rank - k is its place in the merge queue
 *   kept_idx  optional [B][k] int32 out: the kept tokens, ascending
 *   near_tie  optional [B] int32 out: neighbours (p, p+1) of the order with p+1 >= k whose
 *             fp32 gap satisfies (s_p - s_{p+1}) < 1e-4 * |s_p|  (ties the caller may report)
 * -0 equals +0; NaN sorts last and sets LVLM_DEV_NONFINITE (so does an infinity).
 * Errors: INVALID_ARG (NULL score/rank, B<=0, n<=0, k outside [0,n]), UNSUPPORTED (n > 65536;
 * n > 51200 when kept_idx or near_tie is asked for).
 */
lvlm_status lvlm_select_topk(const float* score, int B, int n, int64_t score_stride, int k,
                             int32_t* rank, int32_t* kept_idx, int32_t* near_tie,
                             void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Merge and compaction (Section 3.2.1, paragraph 4): P_new = W_v x P_merged and
 * P_compressed = [P_unmerged, P_new], written inside the full sequence:
 *     [ tokens before the image | kept image tokens, original order | P_new | tokens after ]
 * With r = n-k-1 the sequence shrinks from N to N-r rows; r <= 0 (k >= n-1) leaves every
 * tensor unchanged.  In mode NEAREST_KEPT there is no P_new row and the result has
 * N-(n-k) rows.
 *   hidden      [B][N][C] bf16 (batch stride d->hid_stride_b)
 *   hidden_out  [B][rows after][C] bf16, or NULL (or `hidden` itself) to compact `hidden` in place;
 *               any other overlap with `hidden` is INVALID_ARG
 *   Kc, Vc      optional [B][Hkv][cap][D] bf16: this layer's keys and values, rows 0..N-1
 *               valid; compacted IN PLACE with the same map, the merged row being the same
 *               weighted mean per KV head (pass both or neither)
 *   pos_ids     optional [B][N] int32, compacted in place; P_new takes the id of the most
 *               important merged token
 *   rank        [B][n] int32 from lvlm_select_topk (must be a permutation of 0..n-1)
 *   w_custom    [n-k] fp32 (device) when mode == CUSTOM, else NULL
 *   mass        NEAREST_KEPT only, optional [B][N] fp32 in/out: token masses (NULL = all 1),
 *               compacted in place like pos_ids; a kept token's mass grows by what it absorbs
 *   new_len     optional [B] int32 out: rows after the call
 * Reads d: B,N,C,Hkv,D,cap,i0,n,k,hid_stride_b,out_stride_b,kv_stride_*.
 * Errors: INVALID_ARG (NULL hidden/rank, i0+n>N, k outside [0,n], N>cap with Kc, only one of
 * Kc/Vc, CUSTOM without w_custom, C%8), UNSUPPORTED (D!=128 with Kc; C > 8192 with hidden_out;
 * NEAREST_KEPT without hidden_out), ALIGNMENT, WORKSPACE.
 */
lvlm_status lvlm_merge_compact(void* hidden, void* hidden_out, void* Kc, void* Vc,
                               int32_t* pos_ids, const int32_t* rank, const lvlm_dims* d,
                               lvlm_merge_mode mode, const float* w_custom, float* mass,
                               int32_t* new_len,
                               void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * KV-cache compression (Section 3.2.2, paragraph 2; Appendix A.2: threshold beta = 0.995,
 * layers after Layer 5), independently per (sequence, KV head): among the evictable entries
 *     E = [e_lo[b], min(e_hi[b], len - d->recent))
 * sort by (acc_score descending, index ascending), keep the shortest prefix whose cumulative
 * score reaches beta * (total score of E) - the entry that crosses the threshold is kept -
 * but at most budget - (entries outside E); drop the rest of E.  Survivors keep their order;
 * K, V, acc_score and pos are compacted in place and len is updated.
 * The count is exact: scores are taken in integer units of 2^-24 and beta in parts per
 * million; beta >= 1 disables the threshold (keep all, subject to the budget).
 *   Kc, Vc     [B][Hkv][cap][D] bf16 in/out        acc_score [B][Hkv][cap] fp32 in/out
 *   pos        optional [B][Hkv][cap] int32 in/out len [B][Hkv] int32 in/out
 *   e_lo,e_hi  optional [B] int32 (both or neither); NULL = every entry is evictable
 *   budget     maximum entries per head after the call; <= 0 means no budget
 * The paper's use: e = the image span, beta = 0.995, no budget, once before generation.
 * Periodic use during decoding: e = NULL, beta = 1, budget, d->recent protecting new entries.
 * Reads d: B,Hkv,D,cap,recent,kv_stride_*.
 * Errors: INVALID_ARG (NULL Kc/Vc/acc_score/len, beta outside (0,1], one of e_lo/e_hi),
 * UNSUPPORTED (D!=128, cap > 16384), ALIGNMENT, WORKSPACE.  len > cap sets LVLM_DEV_BOUNDS
 * and that head is left untouched.
 */
lvlm_status lvlm_kv_compress(void* Kc, void* Vc, float* acc_score, int32_t* pos, int32_t* len,
                             const int32_t* e_lo, const int32_t* e_hi, const lvlm_dims* d,
                             float beta, int budget,
                             void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * One decoding step of attention over the (ragged, compressed) cache (Section 3.2.2,
 * paragraph 1: the current token attends to every cached key and value).
 *   o[b,h,:] = softmax(q[b,h,:] . K[b,g,0:len[b,g],:]^T * scale) V[b,g,0:len[b,g],:],  g = h/(H/Hkv)
 *   q        [B][H][D] bf16            out [B][H][D] bf16
 *   Kc, Vc   [B][Hkv][cap][D] bf16     len [B][Hkv] int32
 *   k_new, v_new  optional [B][Hkv][D] bf16 (both or neither): appended at row len before
 *            attending, len += 1.  If len == cap the append is skipped, len stays and
 *            LVLM_DEV_BOUNDS is set.
 *   acc_score optional [B][Hkv][cap] fp32 in/out: entry j receives the probabilities of the
 *            group's query heads, acc_score[b,g,j] += sum_{h in g} p[b,h,j]
 * A head with len == 0 (and no append) outputs zeros.  A head whose len lies outside [0, cap]
 * is skipped: zeros are written, nothing is appended, its len is left alone and
 * LVLM_DEV_BOUNDS is set.
 * d->cache_stable = 1 promises that the operation enqueued on the stream just before this call
 * does not write Kc, Vc or len (true between the layers of a model: the cache of a layer was last
 * written in the previous decoding step; NOT true right after lvlm_kv_compress or
 * lvlm_merge_compact on the same cache).  The kernel then starts fetching the cache while that
 * operation is still draining; q, k_new, v_new and all writes wait for it as always.
 * Workspace: only used when acc_score is given and the cache is so long that the scaled logits of a CTA's
 * own keys do not fit in its shared memory (they are then parked there between the pass over the keys and
 * the update of acc_score); its contents need not be zeroed.
 * Reads d: B,H,Hkv,D,cap,kv_stride_*.
 * Errors: INVALID_ARG, UNSUPPORTED (D!=128, H/Hkv > 8), ALIGNMENT, WORKSPACE.
 */
lvlm_status lvlm_decode_attn(const void* q, void* Kc, void* Vc, int32_t* len,
                             const void* k_new, const void* v_new, float* acc_score,
                             const lvlm_dims* d, float scale, void* out,
                             void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * lvlm_decode_attn without a workspace argument.  The paper has no counterpart: this entry
 * point exists for callers that cannot obtain device scratch memory at all - a plug-in inside a
 * serving engine that owns every byte of device memory in a pool sized at start-up, a binding
 * from a runtime that is handed raw tensor pointers but no allocator, or a decode loop that must
 * never meet the device-wide synchronisation cudaMalloc and cudaFree imply.  It computes exactly
 * what lvlm_decode_attn computes, with the same arguments minus `ws`/`ws_bytes`; inputs and
 * outputs are still the caller's.
 *
 * The scratch is a fixed array of LVLM_STATIC_SCRATCH_BYTES inside the library image: every GPU
 * on which the library is loaded carries it until the process exits.  A problem whose
 * lvlm_workspace_bytes(LVLM_OP_DECODE_ATTN, d) exceeds that size is rejected with
 * LVLM_ERR_WORKSPACE and nothing is enqueued (B * H * cap * 4 bytes are needed; B = 8, H = 32,
 * cap = 1152 takes about 1.2 MiB).
 *
 * The first call on each device looks up the array's device address (with that device current)
 * and remembers it; make that first call outside any stream capture.  No call allocates or frees
 * device memory, here or in a library underneath.
 *
 * All calls on one device share the one array, and it keeps whatever the previous call left in
 * it.  Nothing in it has to start at zero - every word a kernel reads was written earlier in the
 * same call - but two calls that overlap on the GPU (different streams, no ordering between
 * them) race on it and corrupt each other's results.  Keep calls on one stream, or order them.
 * Errors: as lvlm_decode_attn; LVLM_ERR_WORKSPACE when the problem does not fit; LVLM_ERR_CUDA
 * when the address lookup fails.
 */
#define LVLM_STATIC_SCRATCH_BYTES (4u << 20)
lvlm_status lvlm_decode_attn_static(const void* q, void* Kc, void* Vc, int32_t* len,
                                    const void* k_new, const void* v_new, float* acc_score,
                                    const lvlm_dims* d, float scale, void* out,
                                    int32_t* dev_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LVLM_H_ */
