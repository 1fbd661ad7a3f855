"""CPU oracle for LightVLM's token-reduction and KV-cache-compression steps.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
CUDA library has to compute.  Only the tests, the smoke check and the CPU
baseline leg of the benchmark may import it; the product never does, and it
shares no code with the CUDA sources.  Inputs are arrays of values that are
already bf16-representable, widened to float64; every sum is taken in float64;
results are stored as float32 (scores) or rounded once to bf16 (token rows).

Steps, in the paper's order and notation (Section 3.2.1 pyramid token merging,
Section 3.2.2 KV-cache compression, Appendix A.2 settings):

  score_tokens    per-key summed attention A, head-averaged        Sec. 3.2.1 par. 3
  attention_with_scores  the layer's attention itself, returning A  Sec. 3.2.1 par. 3 + footnote
  select_topk     split into P_unmerged / P_merged by A, ordered   Sec. 3.2.1 par. 4
  merge_weights   the weight list W_v                              Sec. 3.2.1 par. 4
  merge_compact   P_new = W_v x P_merged; P_compressed             Sec. 3.2.1 par. 4
  nearest_kept_merge  similarity-merge variant (no paper passage)   --
  kv_compress     sort A, keep prefix reaching beta, drop the rest Sec. 3.2.2 par. 2
  decode_attn     current token attends to every cached K, V       Sec. 3.2.2 par. 1
  pyramid_schedule constant reduction ratio from the final budget  App. A.2

Pins (tests/test_oracle_pins.py): textbook softmax, row-sum and harmonic-number
closed forms for the score; for attention_with_scores its last row against
decode_attn, its column sums against score_tokens, row sums of one and
scipy's logsumexp; brute-force subset enumeration for the selection;
closed-form weights, literal iterated pairwise merging and identities for the
merge; no-op / arg-max / uniform-count closed forms for the compression;
len-1, equal-key and GQA identities for decode attention; the printed stage
counts for the schedule.  ``nearest_kept_merge`` follows a rule the paper does
not define (and argues against); its pins are brute force and mass
conservation only.  What stays unpinned: there is no worked numeric example
in the paper, so agreement with the authors' own tensors is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

LINEAR_RANK, GEOMETRIC, UNIFORM, CUSTOM, NEAREST_KEPT = 0, 1, 2, 3, 4

DEV_NONFINITE = 1


# ----------------------------------------------------------------------------
# bf16 helpers (round-to-nearest-even on the top 16 bits of an fp32)
# ----------------------------------------------------------------------------

def round_bf16(x):
    """Round float64/float32 values to the nearest bf16, returned as float32."""
    x32 = np.asarray(x, dtype=np.float32)
    u = x32.view(np.uint32).astype(np.uint64)
    bias = ((u >> np.uint64(16)) & np.uint64(1)) + np.uint64(0x7FFF)
    r = ((u + bias) & np.uint64(0xFFFF0000)).astype(np.uint32)
    out = r.view(np.float32).copy()
    nan = np.isnan(x32)
    if nan.any():
        out[nan] = np.float32(np.nan)
    return out.reshape(x32.shape)


# ----------------------------------------------------------------------------
# Step 1: importance score  (Section 3.2.1, paragraph 3)
# ----------------------------------------------------------------------------

def score_tokens(Q, K, q_lo, q_hi, i0, n, causal=True, scale=None):
    """Summed attention each image key receives from the query rows of a window.

    Q  [B, q_hi-q_lo, H, D]  query rows of sequence positions q_lo..q_hi-1
    K  [B, Hkv, N, D]        keys of the whole sequence
    Row i (position p = q_lo+i) attends, with softmax over ALL keys it can see
    (j <= p when causal, every key otherwise), and contributes its probability
    of key j to A_head[b,h,j].  Returns
      score      [B, n]       float32: mean over the H query heads (the paper's
                              "averaged attention scores across different heads")
      score_head [B, Hkv, n]  float32: sum over the query heads sharing a KV head
    for the image keys j in [i0, i0+n).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    B, Nq, H, D = Q.shape
    Hkv, N = K.shape[1], K.shape[2]
    assert Nq == q_hi - q_lo and H % Hkv == 0
    G = H // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    pos = np.arange(q_lo, q_hi)
    visible = (np.arange(N)[None, :] <= pos[:, None]) if causal else np.ones((Nq, N), bool)
    s_head = np.zeros((B, H, n), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            logits = (Q[b, :, h, :] @ K[b, h // G].T) * scale           # [Nq, N]
            logits = np.where(visible, logits, -np.inf)
            m = logits.max(axis=1, keepdims=True)
            e = np.exp(logits - m)
            p = e / e.sum(axis=1, keepdims=True)
            s_head[b, h] = p[:, i0:i0 + n].sum(axis=0)
    score = s_head.mean(axis=1)
    score_head = s_head.reshape(B, Hkv, G, n).sum(axis=2)
    return score.astype(np.float32), score_head.astype(np.float32)


def attention_with_scores(Q, K, V, q_lo, q_hi, i0, n, causal=True, scale=None):
    """The attention of a prefill layer, returning alongside its output what the token
    reduction reads from it (Section 3.2.1, paragraph 3 and its footnote: the per-key summed
    scores are a by-product of the attention that runs anyway).

    Q  [B, N, H, D]   query rows of sequence positions 0..N-1
    K, V [B, Hkv, N, D]
    Row p attends with softmax over the keys it sees (j <= p when causal).  Returns a dict:
      out        [B, N, H, D] bf16-rounded float32: softmax(Q K^T scale) V
      lse        [B, H, N]    float32: natural log of each row's sum of exponentials
      score      [B, n], score_head [B, Hkv, n]  float32: the probabilities of the rows
                 q_lo..q_hi-1 summed per image key j in [i0, i0+n), head mean / group sum
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    B, N, H, D = Q.shape
    Hkv = K.shape[1]
    assert K.shape[2] == N and V.shape[:3] == K.shape[:3] and H % Hkv == 0 and 0 <= q_lo < q_hi <= N
    G = H // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    visible = (np.arange(N)[None, :] <= np.arange(N)[:, None]) if causal else np.ones((N, N), bool)
    out = np.zeros((B, N, H, V.shape[3]))
    lse = np.zeros((B, H, N))
    s_head = np.zeros((B, H, n))
    for b in range(B):
        for h in range(H):
            logits = (Q[b, :, h, :] @ K[b, h // G].T) * scale            # [N, N]
            logits = np.where(visible, logits, -np.inf)
            m = logits.max(axis=1, keepdims=True)
            e = np.exp(logits - m)
            z = e.sum(axis=1, keepdims=True)
            p = e / z
            out[b, :, h, :] = p @ V[b, h // G]
            lse[b, h] = (m + np.log(z))[:, 0]
            s_head[b, h] = p[q_lo:q_hi, i0:i0 + n].sum(axis=0)
    return {"out": round_bf16(out), "lse": lse.astype(np.float32),
            "score": s_head.mean(axis=1).astype(np.float32),
            "score_head": s_head.reshape(B, Hkv, G, n).sum(axis=2).astype(np.float32)}


# ----------------------------------------------------------------------------
# Step 2: selection  (Section 3.2.1, paragraph 4: P_unmerged / P_merged)
# ----------------------------------------------------------------------------

def _descending_order(score_row):
    """Indices sorted by (score descending, index ascending); NaN last; -0 == +0."""
    s = np.asarray(score_row, dtype=np.float32).astype(np.float64)
    nan = np.isnan(s)
    s = np.where(nan, 0.0, s)
    # keys, least significant first: index, then score descending, then "is NaN"
    return np.lexsort((np.arange(len(s)), -s, nan))


def select_topk(score, k, tie_rel=1e-4):
    """Total order of the n image tokens by importance.

    score [B, n] float32.  rank[b, j] is the position of token j in the order
    (score descending, lower index first among equals).  Tokens with rank < k form
    P_unmerged; the others, in rank order, form P_merged (most important first,
    "tokens of the least importance at the end of the queue").
    Returns rank [B,n] int32, kept_idx [B,k] int32 ascending, near_tie [B] int32,
    status (bit 0 set if a score was NaN or infinite).
    near_tie counts neighbours (p, p+1) of the order with p+1 >= k whose gap is
    below tie_rel relative, taken in float32:  (s_p - s_{p+1}) < tie_rel * |s_p|.
    """
    score = np.asarray(score, dtype=np.float32)
    B, n = score.shape
    rank = np.zeros((B, n), dtype=np.int32)
    kept = np.zeros((B, k), dtype=np.int32)
    near = np.zeros(B, dtype=np.int32)
    status = 0
    for b in range(B):
        if not np.isfinite(score[b]).all():
            status |= DEV_NONFINITE
        order = _descending_order(score[b])
        rank[b, order] = np.arange(n, dtype=np.int32)
        kept[b] = np.sort(order[:k])
        ss = score[b, order]
        cnt = 0
        for p in range(max(k - 1, 0), n - 1):
            a, c = ss[p], ss[p + 1]
            d = np.float32(a - c)
            t = np.float32(np.float32(tie_rel) * np.abs(a))
            if d < t:
                cnt += 1
        near[b] = cnt
    return rank, kept, near, status


# ----------------------------------------------------------------------------
# Step 3: merge weights and merge  (Section 3.2.1, paragraph 4)
# ----------------------------------------------------------------------------

def merge_weights(mode, r1, custom=None):
    """Normalised weights w[0..r1-1] over P_merged in importance order (p = 0 is the
    most important merged token).  r1 = r + 1 tokens are merged into one.

    LINEAR_RANK  the stated list W_v = {r+1, r, ..., 1}, divided by its sum
    GEOMETRIC    what iterating "merge the last two with equal weights" gives when the
                 merge is a mean: (1/2, 1/4, ..., 2^-r, 2^-r)
    UNIFORM      1/(r+1) each
    CUSTOM       the given list, divided by its sum
    """
    if mode == LINEAR_RANK:
        w = np.arange(r1, 0, -1, dtype=np.float64)
    elif mode == GEOMETRIC:
        w = np.ldexp(1.0, -np.arange(1, r1 + 1, dtype=np.int64)).astype(np.float64)
        if r1 >= 1:
            w[-1] = np.ldexp(1.0, -(r1 - 1)) if r1 > 1 else 1.0
    elif mode == UNIFORM:
        w = np.ones(r1, dtype=np.float64)
    elif mode == CUSTOM:
        w = np.asarray(custom, dtype=np.float64)[:r1].copy()
    else:
        raise ValueError(mode)
    return w / w.sum()


def _merge_rows(rows, w):
    """sum_p w[p] * rows[p] in float64."""
    acc = np.zeros(rows.shape[1:], dtype=np.float64)
    for p in range(rows.shape[0]):
        acc += w[p] * rows[p]
    return acc


def merge_compact(hidden, rank, i0, n, k, mode=LINEAR_RANK, custom=None,
                  Kc=None, Vc=None, pos_ids=None):
    """P_compressed = [P_unmerged, P_new] inside the full sequence.

    hidden [B, N, C]; rank [B, n] from select_topk; image span [i0, i0+n).
    The k tokens with rank < k stay, in their original order; the other r+1 = n-k
    tokens, taken in rank order, are merged into one row P_new = W_v x P_merged,
    which is placed right after the last kept image token; text rows before and
    after the span are untouched.  r = 0 (k >= n-1) returns the input unchanged.
    Kc, Vc [B, Hkv, N, D] (that layer's keys and values) and pos_ids [B, N] follow
    the same map; the merged K/V row is the same weighted mean per KV head, and
    P_new takes the position id of the most important merged token.
    Returns dict(hidden [B,N-r,C], Kc, Vc, pos_ids, new_len [B]); rows are rounded to
    bf16 once.
    """
    hidden = np.asarray(hidden, dtype=np.float64)
    B, N, C = hidden.shape
    r1 = n - k
    r = max(r1 - 1, 0)
    out = {"new_len": np.full(B, N - r, dtype=np.int32)}
    if r == 0:
        out["hidden"] = round_bf16(hidden)
        out["Kc"] = None if Kc is None else round_bf16(Kc)
        out["Vc"] = None if Vc is None else round_bf16(Vc)
        out["pos_ids"] = None if pos_ids is None else np.asarray(pos_ids, dtype=np.int32).copy()
        return out
    w = merge_weights(mode, r1, custom)
    h_out = np.zeros((B, N - r, C), dtype=np.float32)
    K_out = V_out = p_out = None
    if Kc is not None:
        Kc = np.asarray(Kc, dtype=np.float64)
        Vc = np.asarray(Vc, dtype=np.float64)
        K_out = np.zeros((B, Kc.shape[1], N - r, Kc.shape[3]), dtype=np.float32)
        V_out = np.zeros_like(K_out)
    if pos_ids is not None:
        pos_ids = np.asarray(pos_ids, dtype=np.int32)
        p_out = np.zeros((B, N - r), dtype=np.int32)
    for b in range(B):
        rk = np.asarray(rank[b])
        kept = np.nonzero(rk < k)[0]                       # ascending index order
        merged = np.argsort(rk, kind="stable")[k:]         # rank order, most important first
        pre = np.arange(0, i0)
        post = np.arange(i0 + n, N)

        def build(x):                                       # x [N, width] float64
            p_new = _merge_rows(x[i0 + merged], w)
            return np.concatenate([x[pre], x[i0 + kept], p_new[None, :], x[post]], axis=0)

        h_out[b] = round_bf16(build(hidden[b]))
        if Kc is not None:
            for g in range(Kc.shape[1]):
                K_out[b, g] = round_bf16(build(Kc[b, g, :N]))
                V_out[b, g] = round_bf16(build(Vc[b, g, :N]))
        if pos_ids is not None:
            p_out[b] = np.concatenate([pos_ids[b, pre], pos_ids[b, i0 + kept],
                                       pos_ids[b, i0 + merged[:1]], pos_ids[b, post]])
    out.update(hidden=h_out, Kc=K_out, Vc=V_out, pos_ids=p_out)
    return out


def nearest_kept_merge(hidden, rank, i0, n, k, mass=None, Kc=None, Vc=None, pos_ids=None, assign=None):
    """Similarity-merge variant (not in the paper): every dropped image token is merged into
    the kept image token it is most similar to.

    For a dropped token d (rank >= k): a(d) = argmax over kept t of the cosine
    similarity of the hidden rows d and t (lower t wins ties).  Each kept t becomes the
    mass-weighted mean of itself and the tokens assigned to it, added in ascending
    token order; masses default to 1.  Output has the k kept image tokens only (no
    extra row): length N - (n - k).  That layer's Kc, Vc [B, Hkv, N, D] follow the same
    assignment and masses per KV head; pos_ids [B, N] keep the kept tokens' ids.
    ``assign`` [B, n-k], when given, replaces the argmax (a test that has verified a
    near-tie continues from the other side's choice).
    Returns dict(hidden, assign [B, n-k] (index into the ascending kept list, dropped
    tokens in ascending index order), sim_best / sim_second [B, n-k] (cosine of the
    chosen and of the runner-up kept token), mass [B, N-(n-k)] or None, Kc, Vc,
    pos_ids, new_len).
    """
    hidden = np.asarray(hidden, dtype=np.float64)
    B, N, C = hidden.shape
    r = n - k
    h_out = np.zeros((B, N - r, C), dtype=np.float32)
    a_out = np.zeros((B, r), dtype=np.int32)
    best = np.zeros((B, r), dtype=np.float64)
    second = np.full((B, r), -np.inf, dtype=np.float64)
    m_out = None if mass is None else np.zeros((B, N - r), dtype=np.float32)
    K_out = V_out = p_out = None
    if Kc is not None:
        Kc = np.asarray(Kc, dtype=np.float64)
        Vc = np.asarray(Vc, dtype=np.float64)
        K_out = np.zeros((B, Kc.shape[1], N - r, Kc.shape[3]), dtype=np.float32)
        V_out = np.zeros_like(K_out)
    if pos_ids is not None:
        pos_ids = np.asarray(pos_ids, dtype=np.int32)
        p_out = np.zeros((B, N - r), dtype=np.int32)
    for b in range(B):
        rk = np.asarray(rank[b])
        kept = np.nonzero(rk < k)[0]
        drop = np.nonzero(rk >= k)[0]
        x = hidden[b, i0:i0 + n]
        nrm = np.sqrt((x * x).sum(axis=1))
        nrm = np.where(nrm > 0, nrm, 1.0)
        m = np.ones(n) if mass is None else np.asarray(mass[b, i0:i0 + n], dtype=np.float64)
        den = m[kept].copy()
        for q, d in enumerate(drop):
            cos = (x[kept] @ x[d]) / (nrm[kept] * nrm[d]) if k > 0 else np.zeros(0)
            t = int(np.argmax(cos)) if assign is None else int(assign[b][q])   # first maximum = lowest index
            a_out[b, q] = t
            best[b, q] = cos[t]
            if k > 1:
                second[b, q] = np.max(np.delete(cos, t))
            den[t] += m[d]

        def merged(rows):                                   # rows [n, width] float64 -> [k, width]
            num = rows[kept] * m[kept, None]
            for q, d in enumerate(drop):
                num[a_out[b, q]] += m[d] * rows[d]
            return num / den[:, None]

        h_out[b] = round_bf16(np.concatenate([hidden[b, :i0], merged(x), hidden[b, i0 + n:]], axis=0))
        if Kc is not None:
            for g in range(Kc.shape[1]):
                K_out[b, g] = round_bf16(np.concatenate(
                    [Kc[b, g, :i0], merged(Kc[b, g, i0:i0 + n]), Kc[b, g, i0 + n:N]], axis=0))
                V_out[b, g] = round_bf16(np.concatenate(
                    [Vc[b, g, :i0], merged(Vc[b, g, i0:i0 + n]), Vc[b, g, i0 + n:N]], axis=0))
        if pos_ids is not None:
            p_out[b] = np.concatenate([pos_ids[b, :i0], pos_ids[b, i0 + kept], pos_ids[b, i0 + n:]])
        if mass is not None:
            mm = np.asarray(mass[b], dtype=np.float64)
            m_out[b] = np.concatenate([mm[:i0], den, mm[i0 + n:]]).astype(np.float32)
    return {"hidden": h_out, "assign": a_out, "sim_best": best, "sim_second": second, "mass": m_out,
            "Kc": K_out, "Vc": V_out, "pos_ids": p_out, "new_len": np.full(B, N - r, dtype=np.int32)}


# ----------------------------------------------------------------------------
# Step 5: KV-cache compression  (Section 3.2.2, paragraph 2; Appendix A.2)
# ----------------------------------------------------------------------------

SCORE_UNIT_BITS = 24          # scores are counted in integer units of 2^-24
BETA_DENOM = 1_000_000        # beta is taken in parts per million


def kv_keep_count(scores_sorted, beta):
    """Length of the shortest prefix of A_des whose cumulative score reaches beta times
    the total; the token that crosses the threshold is kept.  beta >= 1 keeps all.
    Scores are first quantised to integer units of 2^-24 and the test
    cum * 10^6 >= beta_ppm * total is made in exact integer arithmetic."""
    m = len(scores_sorted)
    beta_ppm = int(np.rint(np.float64(np.float32(beta)) * BETA_DENOM))
    if beta_ppm >= BETA_DENOM:
        return m
    q = []
    for s in scores_sorted:
        s = float(np.float32(s))
        if not np.isfinite(s) or s < 0:
            s = 0.0
        q.append(int(np.rint(np.ldexp(s, SCORE_UNIT_BITS))))
    total = sum(q)
    cum = 0
    for c in range(m):
        cum += q[c]
        if cum * BETA_DENOM >= beta_ppm * total:
            return c + 1
    return m


def kv_compress(Kc, Vc, acc_score, length, e_lo=None, e_hi=None, beta=1.0,
                budget=None, recent=0, pos=None):
    """Per (batch, KV head) and independently of the other heads: among the evictable
    entries E = [e_lo[b], min(e_hi[b], len - recent)) sort by (score descending, index
    ascending), keep the shortest prefix whose cumulative score reaches beta * (total
    score of E), but no more than budget - (entries outside E); discard the rest of E.
    Survivors keep their original order.  Entries outside E always stay.

    Kc, Vc [B, Hkv, cap, D]; acc_score [B, Hkv, cap] float32; length [B, Hkv] int.
    Returns dict(Kc, Vc, acc_score, pos, len, keep_idx[b][g] = surviving indices).
    Rows at or beyond the new length are returned unchanged from the input.
    """
    Kc = np.array(Kc, dtype=np.float32)
    Vc = np.array(Vc, dtype=np.float32)
    acc = np.array(acc_score, dtype=np.float32)
    length = np.asarray(length, dtype=np.int64)
    B, Hkv = length.shape
    new_len = np.zeros((B, Hkv), dtype=np.int32)
    pos_out = None if pos is None else np.array(pos, dtype=np.int32)
    keep_all = [[None] * Hkv for _ in range(B)]
    for b in range(B):
        for g in range(Hkv):
            ln = int(length[b, g])
            lo = 0 if e_lo is None else int(e_lo[b])
            hi = ln if e_hi is None else int(e_hi[b])
            hi = min(hi, ln - recent)
            lo = min(max(lo, 0), ln)
            hi = max(hi, lo)
            E = np.arange(lo, hi)
            s = acc[b, g, lo:hi]
            order = _descending_order(s)
            k_beta = kv_keep_count(s[order], beta)
            kc = k_beta
            if budget is not None:
                kc = min(kc, budget - (ln - len(E)))
            kc = min(max(kc, 0), len(E))
            keep = np.concatenate([np.arange(0, lo), np.sort(E[order[:kc]]), np.arange(hi, ln)])
            keep_all[b][g] = keep
            m = len(keep)
            Kc[b, g, :m] = Kc[b, g, keep]
            Vc[b, g, :m] = Vc[b, g, keep]
            acc[b, g, :m] = acc[b, g, keep]
            if pos_out is not None:
                pos_out[b, g, :m] = pos_out[b, g, keep]
            new_len[b, g] = m
    return {"Kc": Kc, "Vc": Vc, "acc_score": acc, "pos": pos_out, "len": new_len,
            "keep_idx": keep_all}


# ----------------------------------------------------------------------------
# Step 6: decode attention over the (ragged) cache  (Section 3.2.2, paragraph 1)
# ----------------------------------------------------------------------------

def decode_attn(q, Kc, Vc, length, k_new=None, v_new=None, acc_score=None, scale=None):
    """One generated token attends to every cached key and value of its KV head.

    q [B, H, D]; Kc, Vc [B, Hkv, cap, D]; length [B, Hkv] (ragged).  When k_new, v_new
    [B, Hkv, D] are given they are appended at row len first and len grows by one.
    o[b,h] = softmax(q[b,h] . K[b,g,0:len]^T * scale) V[b,g,0:len],  g = h // G.
    acc_score [B, Hkv, cap] (optional) receives, per cached entry, the probabilities
    summed over the query heads of the group; an appended entry starts from zero.
    Returns dict(out [B,H,D] bf16-rounded float32, Kc, Vc, len, acc_score).
    """
    q = np.asarray(q, dtype=np.float64)
    Kc = np.array(Kc, dtype=np.float32)
    Vc = np.array(Vc, dtype=np.float32)
    length = np.array(length, dtype=np.int32)
    B, H, D = q.shape
    Hkv = Kc.shape[1]
    G = H // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    acc = None if acc_score is None else np.array(acc_score, dtype=np.float32)
    out = np.zeros((B, H, D), dtype=np.float64)
    for b in range(B):
        for g in range(Hkv):
            ln = int(length[b, g])
            if k_new is not None:
                Kc[b, g, ln] = np.asarray(k_new[b, g], dtype=np.float32)
                Vc[b, g, ln] = np.asarray(v_new[b, g], dtype=np.float32)
                if acc is not None:
                    acc[b, g, ln] = 0.0                    # a new entry starts with no score
                ln += 1
                length[b, g] = ln
            Kd = Kc[b, g, :ln].astype(np.float64)
            Vd = Vc[b, g, :ln].astype(np.float64)
            psum = np.zeros(ln, dtype=np.float64)
            for h in range(g * G, (g + 1) * G):
                logits = (Kd @ q[b, h]) * scale
                e = np.exp(logits - logits.max())
                p = e / e.sum()
                out[b, h] = p @ Vd
                psum += p
            if acc is not None:
                acc[b, g, :ln] = (acc[b, g, :ln].astype(np.float64) + psum).astype(np.float32)
    return {"out": round_bf16(out), "Kc": Kc, "Vc": Vc, "len": length, "acc_score": acc}


# ----------------------------------------------------------------------------
# Pyramid schedule  (Appendix A.2: constant token-reduction ratio set by the budget)
# ----------------------------------------------------------------------------

def pyramid_schedule(n, final_ratio, stages):
    """Image-token counts after each of ``stages`` reductions with a constant per-stage
    keep ratio rho = final_ratio^(1/stages):  M_s = floor(n * final_ratio^(s/stages) + 1/2)."""
    return [int(np.floor(n * final_ratio ** (s / stages) + 0.5)) for s in range(1, stages + 1)]
