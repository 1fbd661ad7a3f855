"""Pins for the CPU oracle: closed forms, invariants, brute force and library routines
that fix what each oracle function must return without consulting the oracle itself."""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.special

from oracle import lvlm_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    return O.round_bf16(np.asarray(x, dtype=np.float64)).astype(np.float64)


def rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ bf16 rounding
def test_round_bf16_known_values():
    # 1 + 2^-8 is exactly half way between bf16 neighbours 1.0 and 1.0078125: ties to even
    assert O.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == np.float32(1.0)
    assert O.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == np.float32(1.015625)
    assert O.round_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -20]))[0] == np.float32(1.0078125)
    assert O.round_bf16(np.array([-3.0]))[0] == np.float32(-3.0)
    v = O.round_bf16(rng(0).normal(size=1000))
    assert np.all((v.view(np.uint32) & 0xFFFF) == 0)


# ------------------------------------------------------------------ score
def test_score_single_row_is_softmax():
    r = rng(1)
    N, D = 37, 16
    Q = bf16(r.normal(size=(1, 1, 1, D)))
    K = bf16(r.normal(size=(1, 1, N, D)))
    scale = 0.37
    s, sh = O.score_tokens(Q, K, q_lo=N - 1, q_hi=N, i0=5, n=20, causal=False, scale=scale)
    ref = scipy.special.softmax((K[0, 0] @ Q[0, 0, 0]) * scale)
    np.testing.assert_allclose(s[0], ref[5:25], rtol=1e-6)
    np.testing.assert_allclose(sh[0, 0], ref[5:25], rtol=1e-6)
    # causal with the last row sees every key: same answer
    s2, _ = O.score_tokens(Q, K, q_lo=N - 1, q_hi=N, i0=5, n=20, causal=True, scale=scale)
    np.testing.assert_allclose(s2, s, rtol=1e-7)


def test_score_rows_sum_to_number_of_rows():
    r = rng(2)
    B, N, H, D = 2, 29, 4, 8
    Q = bf16(r.normal(size=(B, N, H, D)))
    K = bf16(r.normal(size=(B, H, N, D)))
    for causal in (True, False):
        s, sh = O.score_tokens(Q, K, 0, N, 0, N, causal=causal)
        np.testing.assert_allclose(sh.sum(axis=2), N, rtol=1e-6)       # per head
        np.testing.assert_allclose(s.sum(axis=1), N, rtol=1e-6)        # head mean
    s, sh = O.score_tokens(Q, K, 0, N, 0, N, causal=True)
    assert np.all(sh[:, :, 0] >= 1.0)     # row 0 gives key 0 all of its mass
    # window of rows 10..19 only: the sum over all keys is the number of window rows
    s, _ = O.score_tokens(Q[:, 10:20], K, 10, 20, 0, N, causal=True)
    np.testing.assert_allclose(s.sum(axis=1), 10, rtol=1e-6)
    # causal: keys after the window's last row receive nothing
    assert np.all(s[:, 20:] == 0)


def test_score_equal_keys_harmonic_closed_form():
    N, D, H = 23, 8, 2
    r = rng(3)
    Q = bf16(r.normal(size=(1, N, H, D)))
    K = np.tile(bf16(r.normal(size=(1, 1, 1, D))), (1, H, N, 1))
    s, _ = O.score_tokens(Q, K, 0, N, 0, N, causal=True)
    Hn = np.cumsum(1.0 / np.arange(1, N + 1))
    expect = np.array([Hn[N - 1] - (Hn[j - 1] if j > 0 else 0.0) for j in range(N)])
    np.testing.assert_allclose(s[0], expect, rtol=1e-6)


def test_score_gqa_group_mapping_and_head_mean():
    r = rng(4)
    B, N, H, Hkv, D = 1, 12, 6, 2, 8
    Q = bf16(r.normal(size=(B, N, H, D)))
    K = bf16(r.normal(size=(B, Hkv, N, D)))
    K[0, 1] = 0.0            # heads 3,4,5 see equal keys -> uniform over visible keys
    s, sh = O.score_tokens(Q, K, 0, N, 0, N, causal=True)
    Hn = np.cumsum(1.0 / np.arange(1, N + 1))
    uni = np.array([Hn[N - 1] - (Hn[j - 1] if j > 0 else 0.0) for j in range(N)])
    np.testing.assert_allclose(sh[0, 1], 3 * uni, rtol=1e-6)
    # the head mean is (sum over KV groups of the group sums) / H
    np.testing.assert_allclose(s[0], sh[0].sum(axis=0) / H, rtol=1e-6)
    # independent per-head recomputation through the library softmax
    acc = np.zeros(N)
    for h in range(3):
        lg = (Q[0, :, h] @ K[0, 0].T) / math.sqrt(D)
        lg = np.where(np.tril(np.ones((N, N), bool)), lg, -np.inf)
        acc += scipy.special.softmax(lg, axis=1).sum(axis=0)
    np.testing.assert_allclose(sh[0, 0], acc, rtol=1e-6)


def test_score_planted_keys_dominate():
    r = rng(5)
    N, n, D = 80, 64, 128
    Q = bf16(r.normal(size=(1, N, 2, D)))
    K = bf16(r.normal(size=(1, 2, N, D)))
    u = np.ones(D) / math.sqrt(D)
    Q = bf16(Q + 4.0 * u)
    planted = [3, 17, 40]
    K[0, :, planted] = bf16(K[0, :, planted] + 16.0 * u)
    s, _ = O.score_tokens(Q[:, n:], K, n, N, 0, n, causal=True)
    top3 = set(np.argsort(-s[0])[:3].tolist())
    assert top3 == set(planted)
    assert s[0, planted].sum() > 0.8 * s[0].sum()


# ------------------------------------------------------------------ select
@pytest.mark.parametrize("seed", range(6))
def test_select_bruteforce_subsets(seed):
    r = rng(100 + seed)
    n = int(r.integers(1, 11))
    # few distinct values => many ties
    score = r.integers(0, 4, size=(1, n)).astype(np.float32) * np.float32(0.25)
    for k in range(0, n + 1):
        rank, kept, _, status = O.select_topk(score, k)
        assert status == 0
        best = None
        for sub in itertools.combinations(range(n), k):
            key = (-float(np.sum(score[0, list(sub)], dtype=np.float64)), sub)
            if best is None or key < best:
                best = key
        assert tuple(kept[0].tolist()) == best[1]
        # counting definition of the rank (a different algorithm from sorting)
        for j in range(n):
            cnt = sum(1 for i in range(n)
                      if score[0, i] > score[0, j] or (score[0, i] == score[0, j] and i < j))
            assert rank[0, j] == cnt
        assert sorted(rank[0].tolist()) == list(range(n))


def test_select_all_equal_and_permutation():
    rank, kept, near, _ = O.select_topk(np.full((2, 9), 0.5, np.float32), 4)
    assert kept.tolist() == [[0, 1, 2, 3]] * 2
    assert rank.tolist() == [list(range(9))] * 2
    assert near.tolist() == [5, 5]          # pairs (3,4) .. (7,8) all have zero gap
    r = rng(7)
    s = r.random(size=(1, 50)).astype(np.float32)
    perm = r.permutation(50)
    rank, kept, _, _ = O.select_topk(s, 20)
    rank_p, kept_p, _, _ = O.select_topk(s[:, perm], 20)
    assert np.array_equal(rank_p[0], rank[0][perm])
    assert set(perm[kept_p[0]].tolist()) == set(kept[0].tolist())


def test_select_nonfinite_and_signed_zero():
    s = np.array([[0.0, np.nan, -0.0, 1.0, np.inf]], np.float32)
    rank, kept, _, status = O.select_topk(s, 2)
    assert status & O.DEV_NONFINITE
    assert rank[0].tolist() == [2, 4, 3, 1, 0]      # inf, 1, +0 (idx 0), -0 (idx 2), NaN last
    assert kept[0].tolist() == [3, 4]
    # NaN comes strictly after a genuine -inf, whatever their indices
    s = np.array([[np.nan, -np.inf, 2.0]], np.float32)
    rank, _, _, _ = O.select_topk(s, 1)
    assert rank[0].tolist() == [2, 1, 0]


def test_near_tie_counts_only_dropped_side():
    s = np.array([[10.0, 9.0, 8.0, 8.0 * (1 - 5e-5), 1.0, 1.0]], np.float32)
    _, _, near, _ = O.select_topk(s, 3)         # pairs (2,3) straddles, (3,4), (4,5)
    assert near[0] == 2
    _, _, near, _ = O.select_topk(s, 5)         # only pair (4,5)
    assert near[0] == 1


# ------------------------------------------------------------------ merge weights / merge
def test_weights_closed_forms():
    for r1 in (1, 2, 3, 7, 289):
        w = O.merge_weights(O.LINEAR_RANK, r1)
        r = r1 - 1
        expect = np.array([(r + 1 - p) / ((r + 1) * (r + 2) / 2) for p in range(r1)])
        np.testing.assert_allclose(w, expect, rtol=1e-14)
        for mode in (O.LINEAR_RANK, O.GEOMETRIC, O.UNIFORM):
            assert abs(O.merge_weights(mode, r1).sum() - 1.0) < 1e-15
    np.testing.assert_allclose(O.merge_weights(O.LINEAR_RANK, 2), [2 / 3, 1 / 3])
    np.testing.assert_allclose(O.merge_weights(O.GEOMETRIC, 4), [0.5, 0.25, 0.125, 0.125])
    np.testing.assert_allclose(O.merge_weights(O.CUSTOM, 3, [1, 1, 2]), [0.25, 0.25, 0.5])


def test_geometric_equals_literal_iterated_pairwise_merging():
    r = rng(8)
    for r1 in (1, 2, 5, 11):
        rows = r.normal(size=(r1, 6))
        queue = [row.copy() for row in rows]           # most important first
        while len(queue) > 1:                          # merge the last two, equal weights
            b = queue.pop()
            a = queue.pop()
            queue.append(0.5 * (a + b))
        w = O.merge_weights(O.GEOMETRIC, r1)
        np.testing.assert_allclose((w[:, None] * rows).sum(axis=0), queue[0], rtol=1e-12)


def _simple_case(N=20, i0=3, n=12, C=16, seed=9):
    r = rng(seed)
    hidden = bf16(r.normal(size=(1, N, C)))
    score = r.random(size=(1, n)).astype(np.float32)
    return hidden, score


def test_merge_one_hot_rows_give_the_weight_vector():
    n, k = 8, 3
    hidden = np.zeros((1, n, n))
    hidden[0] = np.eye(n)
    score = np.array([[0.9, 0.1, 0.8, 0.2, 0.7, 0.3, 0.05, 0.6]], np.float32)
    rank, kept, _, _ = O.select_topk(score, k)
    out = O.merge_compact(hidden, rank, 0, n, k)
    assert kept[0].tolist() == [0, 2, 4]
    # dropped in importance order: 7 (.6), 5 (.3), 3 (.2), 1 (.1), 6 (.05): weights 5..1 / 15
    expect = np.zeros(n)
    for p, j in enumerate([7, 5, 3, 1, 6]):
        expect[j] = (5 - p) / 15.0
    assert out["hidden"].shape == (1, k + 1, n)
    np.testing.assert_array_equal(out["hidden"][0, k], O.round_bf16(expect))
    np.testing.assert_array_equal(out["hidden"][0, :k], hidden[0, [0, 2, 4]].astype(np.float32))


def test_merge_r1_is_two_thirds_one_third_and_constant_rows():
    hidden = np.zeros((1, 3, 4))
    hidden[0, 0], hidden[0, 1], hidden[0, 2] = 8.0, 2.0, 5.0
    score = np.array([[0.1, 0.5, 0.3]], np.float32)     # order: 1, 2, 0
    rank, _, _, _ = O.select_topk(score, 1)
    out = O.merge_compact(hidden, rank, 0, 3, 1)
    np.testing.assert_allclose(out["hidden"][0, 1], (2 * 5.0 + 8.0) / 3, rtol=4e-3)
    assert out["hidden"].shape[1] == 2 and out["new_len"][0] == 2
    const = np.full((1, 10, 5), 1.5)
    rank, _, _, _ = O.select_topk(rng(1).random((1, 10)).astype(np.float32), 4)
    for mode in (O.LINEAR_RANK, O.GEOMETRIC, O.UNIFORM):
        o = O.merge_compact(const, rank, 0, 10, 4, mode=mode)
        assert np.all(o["hidden"] == 1.5)


def test_compact_identity_layout_and_invariants():
    N, i0, n, C = 20, 3, 12, 16
    hidden, score = _simple_case(N, i0, n, C)
    pos = np.arange(N, dtype=np.int32)[None] * 3 + 1
    Kc = bf16(rng(10).normal(size=(1, 2, N, 8)))
    Vc = bf16(rng(11).normal(size=(1, 2, N, 8)))
    # keep 100 %: k = n and k = n-1 both return the input unchanged
    for k in (n, n - 1):
        rank, _, _, _ = O.select_topk(score, k)
        out = O.merge_compact(hidden, rank, i0, n, k, Kc=Kc, Vc=Vc, pos_ids=pos)
        np.testing.assert_array_equal(out["hidden"], hidden.astype(np.float32))
        np.testing.assert_array_equal(out["Kc"], Kc.astype(np.float32))
        np.testing.assert_array_equal(out["pos_ids"], pos)
        assert out["new_len"][0] == N
    k = 5
    r = n - k - 1
    rank, kept, _, _ = O.select_topk(score, k)
    out = O.merge_compact(hidden, rank, i0, n, k, Kc=Kc, Vc=Vc, pos_ids=pos)
    h = out["hidden"]
    assert h.shape == (1, N - r, C) and out["new_len"][0] == N - r      # |P_compressed| = N - r
    np.testing.assert_array_equal(h[0, :i0], hidden[0, :i0].astype(np.float32))
    np.testing.assert_array_equal(h[0, i0 + k + 1:], hidden[0, i0 + n:].astype(np.float32))
    np.testing.assert_array_equal(h[0, i0:i0 + k], hidden[0, i0 + kept[0]].astype(np.float32))
    p = out["pos_ids"][0]
    assert np.all(np.diff(p[:i0 + k]) > 0) and np.all(np.diff(p[i0 + k + 1:]) > 0)
    order = np.argsort(rank[0])
    assert p[i0 + k] == pos[0, i0 + order[k]]           # merged row: id of its heaviest member
    # merged K row of head 1 equals the closed-form weighted mean
    w = np.arange(r + 1, 0, -1) / ((r + 1) * (r + 2) / 2)
    expect = (w[:, None] * Kc[0, 1, i0 + order[k:]]).sum(axis=0)
    np.testing.assert_array_equal(out["Kc"][0, 1, i0 + k], O.round_bf16(expect))
    np.testing.assert_array_equal(out["Vc"][0, 0, i0:i0 + k], Vc[0, 0, i0 + kept[0]].astype(np.float32))


def test_nearest_kept_bruteforce_and_mass_conservation():
    r = rng(12)
    N, i0, n, C, k = 14, 2, 9, 6, 4
    hidden = bf16(r.normal(size=(1, N, C)))
    score = r.random((1, n)).astype(np.float32)
    rank, kept, _, _ = O.select_topk(score, k)
    mass = np.ones((1, N), np.float32)
    out = O.nearest_kept_merge(hidden, rank, i0, n, k, mass=mass)
    assert out["hidden"].shape == (1, N - (n - k), C)
    np.testing.assert_allclose(out["mass"][0, i0:i0 + k].sum(), n)       # total mass conserved
    x = hidden[0, i0:i0 + n]
    drop = [j for j in range(n) if rank[0, j] >= k]
    # brute force with the textbook cosine from scipy's distance module
    from scipy.spatial.distance import cosine
    num = {t: x[t].copy() for t in kept[0]}
    cnt = {t: 1 for t in kept[0]}
    for q, d in enumerate(drop):
        best = min(kept[0], key=lambda t: (cosine(x[d], x[t]), t))
        assert kept[0][out["assign"][0, q]] == best
        num[best] += x[d]
        cnt[best] += 1
    for q, t in enumerate(kept[0]):
        np.testing.assert_array_equal(out["hidden"][0, i0 + q], O.round_bf16(num[t] / cnt[t]))
    # mass-weighted total of the image rows is conserved up to bf16 rounding
    tot_in = x.sum(axis=0)
    tot_out = (out["hidden"][0, i0:i0 + k].astype(np.float64) * out["mass"][0, i0:i0 + k, None]).sum(axis=0)
    np.testing.assert_allclose(tot_out, tot_in, atol=0.1)
    # K, V and the position ids follow the same assignment: a cache that equals the hidden states
    # comes out equal to them; a forced assignment is obeyed; the runner-up is never more similar
    pos = np.arange(N, dtype=np.int32)[None]
    kv = O.nearest_kept_merge(hidden, rank, i0, n, k, mass=mass, Kc=hidden[:, None], Vc=2 * hidden[:, None], pos_ids=pos)
    np.testing.assert_array_equal(kv["Kc"][0, 0], out["hidden"][0])
    np.testing.assert_array_equal(kv["Vc"][0, 0], O.round_bf16(2 * out["hidden"][0].astype(np.float64)))
    np.testing.assert_array_equal(kv["pos_ids"][0], np.concatenate([pos[0, :i0], i0 + kept[0], pos[0, i0 + n:]]))
    assert (out["sim_best"] >= out["sim_second"]).all()
    forced = np.zeros_like(out["assign"])
    f = O.nearest_kept_merge(hidden, rank, i0, n, k, assign=forced)
    assert (f["assign"] == 0).all() and f["mass"] is None
    np.testing.assert_array_equal(f["hidden"][0, i0], O.round_bf16((x[kept[0][0]] + x[drop].sum(axis=0)) / (1 + len(drop))))


# ------------------------------------------------------------------ kv compression
def _cache(B=2, Hkv=3, cap=24, D=8, seed=13):
    r = rng(seed)
    Kc = bf16(r.normal(size=(B, Hkv, cap, D)))
    Vc = bf16(r.normal(size=(B, Hkv, cap, D)))
    acc = r.random((B, Hkv, cap)).astype(np.float32)
    ln = r.integers(cap // 2, cap + 1, size=(B, Hkv)).astype(np.int32)
    return Kc, Vc, acc, ln


def test_kv_noop_when_beta_one_and_budget_large():
    Kc, Vc, acc, ln = _cache()
    out = O.kv_compress(Kc, Vc, acc, ln, beta=1.0, budget=10 ** 6)
    np.testing.assert_array_equal(out["len"], ln)
    np.testing.assert_array_equal(out["Kc"], Kc.astype(np.float32))
    np.testing.assert_array_equal(out["acc_score"], acc)


def test_kv_budget_one_keeps_argmax_and_heads_are_independent():
    Kc, Vc, acc, ln = _cache()
    out = O.kv_compress(Kc, Vc, acc, ln, beta=1.0, budget=1)
    B, Hkv = ln.shape
    for b in range(B):
        for g in range(Hkv):
            j = int(np.argmax(acc[b, g, :ln[b, g]]))
            assert out["len"][b, g] == 1
            np.testing.assert_array_equal(out["Kc"][b, g, 0], Kc[b, g, j].astype(np.float32))
            np.testing.assert_array_equal(out["Vc"][b, g, 0], Vc[b, g, j].astype(np.float32))
    # permuting the heads permutes the result
    perm = [2, 0, 1]
    out_p = O.kv_compress(Kc[:, perm], Vc[:, perm], acc[:, perm], ln[:, perm], beta=0.7, budget=9)
    out_0 = O.kv_compress(Kc, Vc, acc, ln, beta=0.7, budget=9)
    np.testing.assert_array_equal(out_p["len"], out_0["len"][:, perm])
    np.testing.assert_array_equal(out_p["Kc"], out_0["Kc"][:, perm])


def test_kv_threshold_closed_forms():
    cap, D = 40, 4
    Kc = bf16(rng(14).normal(size=(1, 1, cap, D)))
    Vc = Kc + 1
    ln = np.array([[cap]], np.int32)
    # one entry holds >= beta of the mass => count 1
    acc = np.full((1, 1, cap), 1e-4, np.float32)
    acc[0, 0, 17] = 5.0
    out = O.kv_compress(Kc, Vc, acc, ln, beta=0.995)
    assert out["len"][0, 0] == 1 and out["keep_idx"][0][0].tolist() == [17]
    # uniform scores => ceil(beta * |E|) lowest indices
    acc = np.full((1, 1, cap), 0.25, np.float32)
    for beta, expect in ((0.5, 20), (0.51, 21), (0.995, 40), (0.9, 36), (0.05, 2)):
        out = O.kv_compress(Kc, Vc, acc, ln, beta=beta)
        assert out["len"][0, 0] == expect == math.ceil(round(beta * cap, 9))
        assert out["keep_idx"][0][0].tolist() == list(range(expect))
    # the crossing token is kept: scores .5 .3 .2, beta .6 -> two tokens
    acc = np.zeros((1, 1, cap), np.float32)
    acc[0, 0, :3] = [0.2, 0.5, 0.3]
    out = O.kv_compress(Kc, Vc, acc, np.array([[3]], np.int32), beta=0.6)
    assert out["keep_idx"][0][0].tolist() == [1, 2]
    assert O.kv_keep_count(np.array([0.5, 0.3, 0.2], np.float32), 0.5) == 1
    assert O.kv_keep_count(np.array([0.5, 0.3, 0.2], np.float32), 0.8) == 2
    assert O.kv_keep_count(np.array([0.5, 0.3, 0.2], np.float32), 0.81) == 3


def test_kv_evictable_range_budget_and_recent_window():
    Kc, Vc, acc, ln = _cache(B=1, Hkv=2, cap=30, seed=15)
    ln[:] = [[30, 26]]
    e_lo, e_hi = np.array([4]), np.array([20])
    out = O.kv_compress(Kc, Vc, acc, ln, e_lo=e_lo, e_hi=e_hi, beta=0.5)
    for g in range(2):
        keep = out["keep_idx"][0][g]
        L = ln[0, g]
        assert keep[:4].tolist() == [0, 1, 2, 3]                          # before the span
        assert keep[-(L - 20):].tolist() == list(range(20, L))            # after the span
        mid = keep[4:len(keep) - (L - 20)]
        assert np.all(np.diff(keep) > 0)                                  # original order
        s = acc[0, g, 4:20].astype(np.float64)
        got = acc[0, g, mid].astype(np.float64).sum()
        assert got >= 0.5 * s.sum() - 1e-6
        # minimal: dropping the weakest kept one falls below the threshold
        assert got - acc[0, g, mid].min() < 0.5 * s.sum() + 1e-6
        # exactly the top-|mid| entries
        top = np.sort(4 + np.argsort(-s, kind="stable")[:len(mid)])
        assert mid.tolist() == top.tolist()
        np.testing.assert_array_equal(out["Kc"][0, g, :len(keep)], Kc[0, g, keep].astype(np.float32))
        np.testing.assert_array_equal(out["acc_score"][0, g, :len(keep)], acc[0, g, keep])
    # budget with a protected recent window: the last 6 always stay
    out = O.kv_compress(Kc, Vc, acc, ln, beta=1.0, budget=16, recent=6)
    for g in range(2):
        keep = out["keep_idx"][0][g]
        L = ln[0, g]
        assert len(keep) == 16 and keep[-6:].tolist() == list(range(L - 6, L))
        s = acc[0, g, :L - 6]
        top = np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:10])
        assert keep[:10].tolist() == top.tolist()


# ------------------------------------------------------------------ decode attention
# ------------------------------------------------------------------ attention_with_scores
def _bf(r, *shape):
    return O.round_bf16(r.normal(size=shape)).astype(np.float64)


def test_attention_last_row_is_decode_attention_and_rows_sum_to_one():
    r = np.random.default_rng(21)
    B, N, H, Hkv, D = 2, 37, 6, 2, 16
    Q, K, V = _bf(r, B, N, H, D), _bf(r, B, Hkv, N, D), _bf(r, B, Hkv, N, D)
    a = O.attention_with_scores(Q, K, V, 30, N, 3, 20)
    # the last position sees every key: its output is one decode step over the whole cache
    dec = O.decode_attn(Q[:, N - 1], K, V, np.full((B, Hkv), N, np.int32))
    assert np.array_equal(a["out"][:, N - 1], dec["out"])
    # every position p is a decode step over the first p+1 entries
    for p in (0, 1, 17):
        dec = O.decode_attn(Q[:, p], K, V, np.full((B, Hkv), p + 1, np.int32))
        assert np.array_equal(a["out"][:, p], dec["out"])
    # lse is the log of the row's sum of exponentials (library routine), so exp(logit - lse) sums to one
    scale = 1.0 / math.sqrt(D)
    for b, h, p in [(0, 0, 0), (1, 5, 36), (0, 3, 12)]:
        logits = (Q[b, p, h] @ K[b, h // 3, :p + 1].T) * scale
        assert abs(a["lse"][b, h, p] - scipy.special.logsumexp(logits)) < 1e-5
        assert abs(np.exp(logits - a["lse"][b, h, p].astype(np.float64)).sum() - 1.0) < 1e-5


def test_attention_column_sums_are_the_scores_of_the_window():
    r = np.random.default_rng(22)
    B, N, H, Hkv, D = 1, 50, 4, 2, 8
    Q, K, V = _bf(r, B, N, H, D), _bf(r, B, Hkv, N, D), _bf(r, B, Hkv, N, D)
    for (q_lo, q_hi, i0, n) in [(40, 50, 2, 35), (0, 50, 0, 50), (10, 11, 5, 4)]:
        a = O.attention_with_scores(Q, K, V, q_lo, q_hi, i0, n)
        score, head = O.score_tokens(Q[:, q_lo:q_hi], K, q_lo, q_hi, i0, n)
        assert np.array_equal(a["score"], score) and np.array_equal(a["score_head"], head)
    # a transposed operand or a dropped mask shows here: V = identity-like rows give the probabilities back
    Vp = np.zeros((B, Hkv, N, N)); Vp[:, :, np.arange(N), np.arange(N)] = 1.0
    a = O.attention_with_scores(Q, K, Vp, 0, N, 0, N)
    p = a["out"].astype(np.float64)                       # [B, N, H, N]: row p's probabilities, bf16-rounded
    assert np.all(np.triu(p[0, :, 0, :], k=1) == 0.0)      # nothing from the future
    assert np.allclose(p.sum(axis=3), 1.0, atol=2e-2)
    assert np.allclose(p[0].sum(axis=0).mean(axis=0), a["score"][0], rtol=2e-2, atol=2e-3)


def test_decode_closed_forms():
    r = rng(16)
    B, H, Hkv, cap, D = 2, 4, 2, 12, 8
    q = bf16(r.normal(size=(B, H, D)))
    Kc = bf16(r.normal(size=(B, Hkv, cap, D)))
    Vc = bf16(r.normal(size=(B, Hkv, cap, D)))
    one = np.ones((B, Hkv), np.int32)
    out = O.decode_attn(q, Kc, Vc, one)
    for h in range(H):
        np.testing.assert_array_equal(out["out"][:, h], Vc[:, h // 2, 0].astype(np.float32))
    # equal keys => mean of the values
    Ke = np.tile(Kc[:, :, :1], (1, 1, cap, 1))
    ln = np.array([[cap, 7], [5, 9]], np.int32)
    out = O.decode_attn(q, Ke, Vc, ln)
    for b in range(B):
        for h in range(H):
            g = h // 2
            np.testing.assert_array_equal(out["out"][b, h], O.round_bf16(Vc[b, g, :ln[b, g]].mean(axis=0)))
    # library softmax, ragged lengths, accumulated probabilities
    acc = np.zeros((B, Hkv, cap), np.float32)
    out = O.decode_attn(q, Kc, Vc, ln, acc_score=acc, scale=0.3)
    for b in range(B):
        for g in range(Hkv):
            L = ln[b, g]
            ps = np.zeros(L)
            for h in (2 * g, 2 * g + 1):
                p = scipy.special.softmax((Kc[b, g, :L] @ q[b, h]) * 0.3)
                np.testing.assert_allclose(out["out"][b, h], O.round_bf16(p @ Vc[b, g, :L]), rtol=1e-2, atol=1e-3)
                ps += p
            np.testing.assert_allclose(out["acc_score"][b, g, :L], ps, rtol=1e-6)
            assert np.all(out["acc_score"][b, g, L:] == 0)
            np.testing.assert_allclose(out["acc_score"][b, g].sum(), 2.0, rtol=1e-6)   # G per step
    # heads of one group with equal queries give equal outputs
    q2 = q.copy()
    q2[:, 1] = q2[:, 0]
    out = O.decode_attn(q2, Kc, Vc, ln)
    np.testing.assert_array_equal(out["out"][:, 0], out["out"][:, 1])


def test_decode_append_is_visible_to_the_same_step():
    r = rng(17)
    B, H, Hkv, cap, D = 1, 2, 1, 6, 8
    q = bf16(r.normal(size=(B, H, D)))
    Kc = bf16(r.normal(size=(B, Hkv, cap, D)))
    Vc = bf16(r.normal(size=(B, Hkv, cap, D)))
    kn = bf16(r.normal(size=(B, Hkv, D)))
    vn = bf16(r.normal(size=(B, Hkv, D)))
    ln = np.array([[3]], np.int32)
    a = O.decode_attn(q, Kc, Vc, ln, k_new=kn, v_new=vn)
    K2, V2 = Kc.copy(), Vc.copy()
    K2[0, 0, 3], V2[0, 0, 3] = kn[0, 0], vn[0, 0]
    b = O.decode_attn(q, K2, V2, np.array([[4]], np.int32))
    np.testing.assert_array_equal(a["out"], b["out"])
    assert a["len"][0, 0] == 4
    np.testing.assert_array_equal(a["Kc"][0, 0, 3], kn[0, 0].astype(np.float32))
    # an empty cache with an append returns the appended value
    z = O.decode_attn(q, Kc, Vc, np.array([[0]], np.int32), k_new=kn, v_new=vn)
    np.testing.assert_array_equal(z["out"][0, 0], vn[0, 0].astype(np.float32))


# ------------------------------------------------------------------ schedule
def test_schedule_matches_hand_computed_table():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "pyramid_schedule.txt"))
            if ln.strip() and not ln.startswith("#")]
    for n, ratio, *counts in rows:
        got = O.pyramid_schedule(int(n), float(ratio), len(counts))
        assert got == [int(c) for c in counts]
