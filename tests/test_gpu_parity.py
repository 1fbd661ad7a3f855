"""CUDA kernels against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import lvlm_oracle as O
from paper_2509_00419_b200 import binding as L
from paper_2509_00419_b200 import inputs as I
from tests.util import assert_rows_close, assert_scores_close, bf16_cuda, f64, i32

pytestmark = pytest.mark.gpu


def status_tensor():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


# ------------------------------------------------------------------ select
@pytest.mark.parametrize("n", [1, 2, 3, 7, 129, 576, 1000, 2880, 4097, 16384, 40000, 65536])
def test_select_bit_exact(n):
    r = np.random.default_rng(n)
    B = 3 if n < 5000 else (2 if n < 20000 else 1)
    s = r.random((B, n)).astype(np.float32)
    s[-1] = np.round(s[-1] * 8) / 8                    # heavy ties in one sequence
    st = torch.from_numpy(s).cuda()
    extras = n <= 51200                               # kept list and near-tie count: up to 51200 tokens
    for k in sorted({0, 1, n // 2, n - 1, n} & set(range(0, n + 1))):
        rank, kept, near = L.select_topk(st, k, want_near=extras, want_kept=extras)
        o_rank, o_kept, o_near, _ = O.select_topk(s, k)
        assert np.array_equal(i32(rank), o_rank), (n, k)
        if extras:
            assert np.array_equal(i32(kept), o_kept), (n, k)
            assert np.array_equal(i32(near), o_near), (n, k)


def test_select_nonfinite_strided_and_flags():
    s = np.array([[0.0, np.nan, -0.0, 1.0, np.inf, 0.5, -1.0, -np.inf, 9.0, 9.0]], np.float32)
    buf = torch.zeros(2, 16, dtype=torch.float32, device="cuda")
    buf[:, :10] = torch.from_numpy(np.repeat(s, 2, 0)).cuda()
    flag = status_tensor()
    rank, kept, _ = L.select_topk(buf[:, :10], 4, dev_status=flag)
    o_rank, o_kept, _, o_flag = O.select_topk(np.repeat(s, 2, 0), 4)
    assert np.array_equal(i32(rank), o_rank) and np.array_equal(i32(kept), o_kept)
    assert flag.item() == o_flag == L.DEV_NONFINITE


# ------------------------------------------------------------------ merge + compact
CASES = [  # B, N, i0, n, C, k
    (1, 20, 3, 12, 16, 5), (2, 77, 0, 64, 136, 31), (2, 300, 11, 257, 1024, 100),
    (1, 640, 0, 576, 1024, 287), (3, 200, 5, 129, 3584, 0), (1, 133, 4, 129, 264, 127),
    (2, 1500, 16, 1400, 512, 40),
]


def _merge_inputs(B, N, i0, n, C, k, Hkv=2, seed=0):
    r = np.random.default_rng(seed + N)
    hidden = torch.from_numpy(r.normal(size=(B, N, C)).astype(np.float32)).to(torch.bfloat16)
    Kc = torch.from_numpy(r.normal(size=(B, Hkv, N + 7, 128)).astype(np.float32)).to(torch.bfloat16)
    Vc = torch.from_numpy(r.normal(size=(B, Hkv, N + 7, 128)).astype(np.float32)).to(torch.bfloat16)
    score = r.random((B, n)).astype(np.float32)
    pos = (np.arange(N, dtype=np.int32)[None] * 2 + 5).repeat(B, 0)
    rank, _, _, _ = O.select_topk(score, k)
    return hidden, Kc, Vc, pos, rank


def _check_merge(out_h, out_K, out_V, out_pos, new_len, want, N, i0, n, k, Kin, Vin):
    r = max(n - k - 1, 0)
    Nout = N - r
    assert np.array_equal(i32(new_len), want["new_len"])
    got = f64(out_h)[:, :Nout]
    w = want["hidden"].astype(np.float64)
    if r > 0:
        mrow = i0 + k
        keep = np.ones(Nout, bool); keep[mrow] = False
        assert np.array_equal(got[:, keep], w[:, keep]), "moved rows must be bit-identical"
        assert_rows_close(got[:, mrow], w[:, mrow], what="merged hidden row")
    else:
        assert np.array_equal(got, w)
    if out_K is not None:
        gK, gV = f64(out_K), f64(out_V)
        wK, wV = want["Kc"].astype(np.float64), want["Vc"].astype(np.float64)
        if r > 0:
            assert np.array_equal(gK[:, :, :Nout][:, :, keep], wK[:, :, keep])
            assert np.array_equal(gV[:, :, :Nout][:, :, keep], wV[:, :, keep])
            assert_rows_close(gK[:, :, mrow], wK[:, :, mrow], what="merged K row")
            assert_rows_close(gV[:, :, mrow], wV[:, :, mrow], what="merged V row")
        else:
            assert np.array_equal(gK[:, :, :N], wK) and np.array_equal(gV[:, :, :N], wV)
        # rows past the old length are never touched
        assert np.array_equal(gK[:, :, N:], f64(Kin)[:, :, N:])
        assert np.array_equal(gV[:, :, N:], f64(Vin)[:, :, N:])
    if out_pos is not None:
        assert np.array_equal(i32(out_pos)[:, :Nout], want["pos_ids"])


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("mode", [O.LINEAR_RANK, O.GEOMETRIC, O.UNIFORM, O.CUSTOM])
def test_merge_compact_out_of_place(case, mode):
    B, N, i0, n, C, k = case
    hidden, Kc, Vc, pos, rank = _merge_inputs(*case)
    custom = np.random.default_rng(1).random(n - k).astype(np.float32) + 0.1 if mode == O.CUSTOM else None
    want = O.merge_compact(f64(hidden), rank, i0, n, k, mode=mode, custom=custom,
                           Kc=f64(Kc)[:, :, :N], Vc=f64(Vc)[:, :, :N], pos_ids=pos)
    h, Kd, Vd = hidden.cuda(), Kc.cuda(), Vc.cuda()
    pd = torch.from_numpy(pos).cuda()
    flag = status_tensor()
    out, new_len = L.merge_compact(h, torch.from_numpy(rank).cuda(), i0=i0, k=k, mode=mode, Kc=Kd,
                                   Vc=Vd, pos_ids=pd, dev_status=flag,
                                   w_custom=None if custom is None else torch.from_numpy(custom).cuda())
    torch.cuda.synchronize()
    assert flag.item() == 0
    assert torch.equal(h.cpu(), hidden), "out-of-place call must not modify the input"
    _check_merge(out, Kd, Vd, pd, new_len, want, N, i0, n, k, Kc, Vc)


@pytest.mark.parametrize("case", CASES)
def test_merge_compact_in_place_and_deterministic(case):
    B, N, i0, n, C, k = case
    hidden, Kc, Vc, pos, rank = _merge_inputs(*case, seed=3)
    want = O.merge_compact(f64(hidden), rank, i0, n, k, Kc=f64(Kc)[:, :, :N], Vc=f64(Vc)[:, :, :N],
                           pos_ids=pos)
    outs = []
    for _ in range(2):
        h, Kd, Vd = hidden.cuda(), Kc.cuda(), Vc.cuda()
        pd = torch.from_numpy(pos).cuda()
        out, new_len = L.merge_compact(h, torch.from_numpy(rank).cuda(), i0=i0, k=k, Kc=Kd, Vc=Vd,
                                       pos_ids=pd, in_place=True)
        torch.cuda.synchronize()
        _check_merge(out, Kd, Vd, pd, new_len, want, N, i0, n, k, Kc, Vc)
        Nout = int(new_len[0])
        outs.append((out[:, :Nout].cpu(), Kd.cpu(), Vd.cpu()))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b), "results must be bit-reproducible"


def test_merge_keep_all_is_identity():
    B, N, i0, n, C = 2, 50, 4, 40, 64
    for k in (n, n - 1):
        hidden, Kc, Vc, pos, rank = _merge_inputs(B, N, i0, n, C, k)
        h, Kd, Vd = hidden.cuda(), Kc.cuda(), Vc.cuda()
        out, new_len = L.merge_compact(h, torch.from_numpy(rank).cuda(), i0=i0, k=k, Kc=Kd, Vc=Vd)
        assert torch.equal(out.cpu(), hidden) and torch.equal(Kd.cpu(), Kc)
        assert new_len.tolist() == [N, N]


# ------------------------------------------------------------------ score
SCORE_CASES = [  # B, N, i0, n, H, Hkv, q_lo, q_hi, causal
    (1, 96, 0, 64, 2, 2, 64, 96, True),          # text window
    (2, 200, 7, 150, 4, 2, 157, 200, True),      # text window, GQA, prefix
    (1, 130, 3, 100, 6, 2, 0, 130, True),        # all rows (column sums of the causal matrix)
    (1, 130, 3, 100, 3, 1, 0, 130, False),       # all rows, no mask
    (2, 300, 0, 257, 8, 8, 40, 300, True),       # window starting inside the image
    (1, 77, 5, 60, 7, 1, 76, 77, True),          # single row
]


@pytest.mark.parametrize("case", SCORE_CASES)
def test_score_tokens(case):
    B, N, i0, n, H, Hkv, q_lo, q_hi, causal = case
    r = np.random.default_rng(N + H)
    Q = torch.from_numpy(r.normal(size=(B, N, H, 128)).astype(np.float32)).to(torch.bfloat16)
    K = torch.from_numpy(r.normal(size=(B, Hkv, N + 9, 128)).astype(np.float32)).to(torch.bfloat16)
    K[:, :, i0 + 3] *= 3.0
    want, want_head = O.score_tokens(f64(Q)[:, q_lo:q_hi], f64(K)[:, :, :N], q_lo, q_hi, i0, n, causal)
    Qd, Kd = Q.cuda(), K.cuda()
    flag = status_tensor()
    got, got_head = L.score_tokens(Qd[:, q_lo:q_hi], Kd, N=N, i0=i0, n=n, q_lo=q_lo, q_hi=q_hi,
                                   causal=causal, want_head=True, dev_status=flag)
    torch.cuda.synchronize()
    assert flag.item() == 0
    assert_scores_close(f64(got), want, what="score")
    assert_scores_close(f64(got_head), want_head, what="score_head")
    # handing over the rows' log-sum-exp gives the same scores
    Qf, Kf = f64(Q)[:, q_lo:q_hi], f64(K)[:, :, :N]
    G = H // Hkv
    lse = np.zeros((B, H, q_hi - q_lo), np.float32)
    for b in range(B):
        for h in range(H):
            lg = (Qf[b, :, h] @ Kf[b, h // G].T) / np.sqrt(128)
            if causal:
                vis = np.arange(N)[None, :] <= np.arange(q_lo, q_hi)[:, None]
                lg = np.where(vis, lg, -np.inf)
            mx = lg.max(axis=1)
            lse[b, h] = mx + np.log(np.exp(lg - mx[:, None]).sum(axis=1))
    got2, _ = L.score_tokens(Qd[:, q_lo:q_hi], Kd, N=N, i0=i0, n=n, q_lo=q_lo, q_hi=q_hi,
                             causal=causal, lse=torch.from_numpy(lse).cuda())
    assert_scores_close(f64(got2), want, what="score with lse")


# ------------------------------------------------------------------ kv compression
KV_CASES = [  # B, Hkv, cap, beta, budget, recent, use_range
    (2, 3, 64, 0.995, 0, 0, True), (2, 2, 200, 0.9, 0, 0, False), (1, 8, 1024, 1.0, 256, 0, False),
    (3, 2, 1152, 1.0, 1024, 128, False), (2, 4, 333, 0.5, 100, 16, True), (1, 1, 5, 0.7, 0, 0, False),
    (1, 2, 8192, 0.99, 0, 0, True), (1, 2, 9000, 0.97, 4000, 64, False), (2, 2, 2048, 0.995, 0, 0, False),
    (1, 2, 3000, 0.99, 0, 0, False), (2, 2, 4096, 1.0, 2500, 32, True), (2, 3, 1536, 0.98, 700, 8, False),
    (40, 16, 96, 0.9, 40, 4, False), (37, 16, 1100, 0.97, 600, 16, True), (150, 4, 2048, 1.0, 1900, 0, False),
    (75, 8, 2500, 0.99, 0, 0, False), (75, 8, 1024, 0.995, 0, 0, True),
]


@pytest.mark.parametrize("case", KV_CASES)
def test_kv_compress_bit_exact(case):
    B, Hkv, cap, beta, budget, recent, use_range = case
    r = np.random.default_rng(cap)
    Kc = torch.from_numpy(r.normal(size=(B, Hkv, cap, 128)).astype(np.float32)).to(torch.bfloat16)
    Vc = torch.from_numpy(r.normal(size=(B, Hkv, cap, 128)).astype(np.float32)).to(torch.bfloat16)
    acc = (r.random((B, Hkv, cap)) ** 6).astype(np.float32)       # a few entries dominate
    acc[0, 0, : cap // 4] = 0.125                                   # ties
    ln = r.integers(cap // 2, cap + 1, size=(B, Hkv)).astype(np.int32)
    ln[0, 0] = cap
    pos = r.integers(0, 10 ** 6, size=(B, Hkv, cap)).astype(np.int32)
    e_lo = e_hi = None
    if use_range:
        e_lo = r.integers(0, cap // 4, size=B).astype(np.int32)
        e_hi = (e_lo + cap // 2).astype(np.int32)
    # with hundreds of heads (the shapes that get one warp per head) the oracle checks three of the sequences
    sel = np.array([0, B // 2, B - 1]) if B * Hkv >= 500 else np.arange(B)
    want = O.kv_compress(f64(Kc[sel]), f64(Vc[sel]), acc[sel], ln[sel], e_lo=None if e_lo is None else e_lo[sel],
                         e_hi=None if e_hi is None else e_hi[sel], beta=beta,
                         budget=budget if budget > 0 else None, recent=recent, pos=pos[sel])
    Kd, Vd = Kc.cuda(), Vc.cuda()
    ad, ld, pd = torch.from_numpy(acc).cuda(), torch.from_numpy(ln).cuda(), torch.from_numpy(pos).cuda()
    flag = status_tensor()
    L.kv_compress(Kd, Vd, ad, ld, beta=beta, budget=budget, recent=recent, pos=pd, dev_status=flag,
                  e_lo=None if e_lo is None else torch.from_numpy(e_lo).cuda(),
                  e_hi=None if e_hi is None else torch.from_numpy(e_hi).cuda())
    torch.cuda.synchronize()
    assert flag.item() == 0
    assert np.array_equal(i32(ld)[sel], want["len"])
    sel_d = torch.from_numpy(sel).cuda()
    gK, gV, ga, gp = f64(Kd[sel_d]), f64(Vd[sel_d]), ad[sel_d].cpu().numpy(), i32(pd[sel_d])
    for b in range(len(sel)):
        for g in range(Hkv):
            m = want["len"][b, g]
            assert np.array_equal(gK[b, g, :m], want["Kc"][b, g, :m].astype(np.float64)), (b, g)
            assert np.array_equal(gV[b, g, :m], want["Vc"][b, g, :m].astype(np.float64)), (b, g)
            assert np.array_equal(ga[b, g, :m], want["acc_score"][b, g, :m])
            assert np.array_equal(gp[b, g, :m], want["pos"][b, g, :m])


# ------------------------------------------------------------------ decode attention
DEC_CASES = [  # B, H, Hkv, cap, append, with_acc
    (2, 4, 2, 100, False, True), (1, 8, 8, 1024, True, True), (3, 28, 4, 300, True, False),
    (2, 48, 8, 640, True, True), (2, 3, 3, 70, False, False), (1, 32, 8, 1152, True, True),
]


@pytest.mark.parametrize("case", DEC_CASES)
def test_decode_attn(case):
    B, H, Hkv, cap, append, with_acc = case
    r = np.random.default_rng(cap + H)
    q = torch.from_numpy(r.normal(size=(B, H, 128)).astype(np.float32)).to(torch.bfloat16)
    Kc = torch.from_numpy(r.normal(size=(B, Hkv, cap, 128)).astype(np.float32)).to(torch.bfloat16)
    Vc = torch.from_numpy(r.normal(size=(B, Hkv, cap, 128)).astype(np.float32)).to(torch.bfloat16)
    kn = torch.from_numpy(r.normal(size=(B, Hkv, 128)).astype(np.float32)).to(torch.bfloat16)
    vn = torch.from_numpy(r.normal(size=(B, Hkv, 128)).astype(np.float32)).to(torch.bfloat16)
    ln = r.integers(1, cap, size=(B, Hkv)).astype(np.int32)
    ln[0, 0] = cap - 1
    if B * Hkv > 2:
        ln.reshape(-1)[1] = 0 if append else 1
    acc = r.random((B, Hkv, cap)).astype(np.float32) if with_acc else None
    want = O.decode_attn(f64(q), f64(Kc), f64(Vc), ln, k_new=f64(kn) if append else None,
                         v_new=f64(vn) if append else None, acc_score=acc)
    Kd, Vd, ld = Kc.cuda(), Vc.cuda(), torch.from_numpy(ln).cuda()
    ad = torch.from_numpy(acc).cuda() if with_acc else None
    flag = status_tensor()
    out = L.decode_attn(q.cuda(), Kd, Vd, ld, k_new=kn.cuda() if append else None,
                        v_new=vn.cuda() if append else None, acc_score=ad, dev_status=flag)
    torch.cuda.synchronize()
    assert flag.item() == 0
    assert_rows_close(f64(out), want["out"], what="attention output")
    assert np.array_equal(i32(ld), want["len"])
    if append:
        assert np.array_equal(f64(Kd), want["Kc"].astype(np.float64))
        assert np.array_equal(f64(Vd), want["Vc"].astype(np.float64))
    if with_acc:
        ga = ad.cpu().numpy()
        for b in range(B):
            for g in range(Hkv):
                m = want["len"][b, g]
                assert_scores_close(ga[b, g, :m], want["acc_score"][b, g, :m], what="acc_score")
                if not append:
                    assert np.array_equal(ga[b, g, m:], acc[b, g, m:])


def test_decode_append_at_capacity_sets_flag():
    B, H, Hkv, cap = 1, 2, 1, 64
    q = torch.randn(B, H, 128, device="cuda").to(torch.bfloat16)
    Kc = torch.randn(B, Hkv, cap, 128, device="cuda").to(torch.bfloat16)
    Vc = torch.randn(B, Hkv, cap, 128, device="cuda").to(torch.bfloat16)
    kn = torch.randn(B, Hkv, 128, device="cuda").to(torch.bfloat16)
    ld = torch.full((B, Hkv), cap, dtype=torch.int32, device="cuda")
    K0 = Kc.clone()
    flag = status_tensor()
    out = L.decode_attn(q, Kc, Vc, ld, k_new=kn, v_new=kn, dev_status=flag)
    want = O.decode_attn(f64(q), f64(K0), f64(Vc), np.full((B, Hkv), cap, np.int32))
    assert flag.item() == L.DEV_BOUNDS and ld.item() == cap and torch.equal(Kc, K0)
    assert_rows_close(f64(out), want["out"])


# ------------------------------------------------------------------ config 1 end to end
def test_cfg1_pipeline():
    w = I.CFG1
    hidden = I.hidden_states(w)
    pos = torch.arange(w.N, dtype=torch.int32)[None].repeat(w.B, 1)
    Q, K, V = I.layer_qkv(w, 0, pos)
    n, k = w.n, w.stages[0][1] - 1
    q_lo, q_hi = w.i0 + w.n, w.N
    # oracle chain
    o_score, o_head = O.score_tokens(f64(Q)[:, q_lo:q_hi], f64(K), q_lo, q_hi, w.i0, n)
    o_rank, o_kept, _, _ = O.select_topk(o_score, k)
    o_out = O.merge_compact(f64(hidden), o_rank, w.i0, n, k, Kc=f64(K), Vc=f64(V), pos_ids=pos.numpy())
    planted = I.planted_positions(w, 0).numpy()
    assert set(planted.tolist()) <= set(o_kept[0].tolist()), "planted keys are among the kept ones"
    # GPU chain
    Qd, Kd, Vd, hd, pd = Q.cuda(), K.cuda(), V.cuda(), hidden.cuda(), pos.cuda()
    score, head = L.score_tokens(Qd[:, q_lo:q_hi], Kd, N=w.N, i0=w.i0, n=n, q_lo=q_lo, q_hi=q_hi,
                                 want_head=True)
    assert_scores_close(f64(score), o_score, what="cfg1 score")
    rank, kept, near = L.select_topk(score, k, want_near=True)
    g_rank = i32(rank)
    mism = np.nonzero(g_rank != o_rank)
    for b, j in zip(*mism):                       # any disagreement must be a near-tie in the oracle
        other = np.nonzero(o_rank[b] == g_rank[b, j])[0][0]
        a, c = float(o_score[b, j]), float(o_score[b, other])
        assert abs(a - c) <= 1e-4 * max(abs(a), abs(c)), "rank mismatch that is not a near-tie"
    # feed the oracle's rank to isolate merge/compact, then the GPU's own rank end to end
    out, new_len = L.merge_compact(hd, torch.from_numpy(o_rank).cuda(), i0=w.i0, k=k, Kc=Kd, Vc=Vd,
                                   pos_ids=pd)
    _check_merge(out, Kd, Vd, pd, new_len, o_out, w.N, w.i0, n, k, K, V)
    if mism[0].size == 0:
        out2, _ = L.merge_compact(hd, rank, i0=w.i0, k=k)
        assert torch.equal(out2, out)
    # one-layer cache of 1024 entries -> budget 256, then one decode step
    cap = w.cap
    r = np.random.default_rng(0)
    Kc = I.normal_bf16(w.seed, "cfg1/cacheK", (w.B, w.Hkv, cap, 128))
    Vc = I.normal_bf16(w.seed, "cfg1/cacheV", (w.B, w.Hkv, cap, 128))
    qs = I.normal_bf16(w.seed, "cfg1/scoreQ", (w.B, 64, w.H, 128))
    acc0, _ = O.score_tokens(f64(qs), f64(Kc), cap, cap + 64, 0, cap, causal=False)
    _, acc_head = O.score_tokens(f64(qs), f64(Kc), cap, cap + 64, 0, cap, causal=False)
    ln = np.full((w.B, w.Hkv), cap, np.int32)
    o_kv = O.kv_compress(f64(Kc), f64(Vc), acc_head, ln, beta=1.0, budget=w.budget)
    qd = I.normal_bf16(w.seed, "cfg1/decq", (w.B, w.H, 128))
    o_dec = O.decode_attn(f64(qd), o_kv["Kc"], o_kv["Vc"], o_kv["len"], acc_score=o_kv["acc_score"])
    Kd, Vd = Kc.cuda(), Vc.cuda()
    _, g_head = L.score_tokens(qs.cuda(), Kd, N=cap, i0=0, n=cap, q_lo=0, q_hi=64, causal=False,
                               want_head=True)
    assert_scores_close(f64(g_head), acc_head, what="cache scores")
    ad = torch.from_numpy(acc_head).cuda()          # same fp32 scores on both sides
    ld = torch.from_numpy(ln).cuda()
    L.kv_compress(Kd, Vd, ad, ld, beta=1.0, budget=w.budget)
    assert np.array_equal(i32(ld), o_kv["len"]) and int(ld.max()) == w.budget
    m = w.budget
    assert np.array_equal(f64(Kd)[:, :, :m], o_kv["Kc"][:, :, :m].astype(np.float64))
    assert np.array_equal(f64(Vd)[:, :, :m], o_kv["Vc"][:, :, :m].astype(np.float64))
    out = L.decode_attn(qd.cuda(), Kd, Vd, ld, acc_score=ad)
    assert_rows_close(f64(out), o_dec["out"], what="cfg1 decode")
    assert_scores_close(ad.cpu().numpy()[:, :, :m], o_dec["acc_score"][:, :, :m], what="cfg1 acc")


# ------------------------------------------------------------------ nearest-kept merge (variant that is not in the paper)
NK_CASES = [  # B, N, i0, n, C, k, Hkv, with_mass, with_kv
    (1, 40, 3, 30, 64, 7, 1, False, False), (2, 700, 5, 640, 256, 300, 2, True, True),
    (1, 1500, 0, 1400, 200, 130, 2, False, True), (3, 333, 2, 300, 1024, 299, 1, True, False),
    (1, 520, 8, 500, 3584, 1, 4, True, True), (2, 600, 0, 600, 512, 600, 2, False, True),
]


@pytest.mark.parametrize("case", NK_CASES)
def test_merge_nearest_kept(case):
    B, N, i0, n, C, k, Hkv, with_mass, with_kv = case
    r = np.random.default_rng(N + C)
    # clustered rows so that similarities are well separated, plus noise
    cent = r.normal(size=(24, C))
    hidden = cent[r.integers(0, 24, size=(B, N))] + 0.4 * r.normal(size=(B, N, C))
    hidden = torch.from_numpy(hidden.astype(np.float32)).to(torch.bfloat16)
    score = r.random((B, n)).astype(np.float32)
    rank, _, _, _ = O.select_topk(score, k)
    pos = np.tile(np.arange(N, dtype=np.int32) * 3, (B, 1))
    mass = (1 + r.integers(0, 4, size=(B, N))).astype(np.float32) if with_mass else None
    Kc = torch.from_numpy(r.normal(size=(B, Hkv, N, 128)).astype(np.float32)).to(torch.bfloat16) if with_kv else None
    Vc = torch.from_numpy(r.normal(size=(B, Hkv, N, 128)).astype(np.float32)).to(torch.bfloat16) if with_kv else None
    ref = O.nearest_kept_merge(f64(hidden), rank, i0, n, k, mass=mass)

    hd, rd = hidden.cuda(), torch.from_numpy(rank).cuda()
    Kd, Vd = (Kc.cuda(), Vc.cuda()) if with_kv else (None, None)
    pd = torch.from_numpy(pos).cuda()
    md = torch.from_numpy(mass).cuda() if with_mass else None
    d = L.merge_dims(hd, rd, i0=i0, k=k, Kc=Kd)
    d.merge_mode = L.W_NEAREST_KEPT
    ws = L.alloc_workspace(L.OP_MERGE_COMPACT, d, hd.device)
    flag = status_tensor()
    out, new_len = L.merge_compact(hd, rd, i0=i0, k=k, mode=L.W_NEAREST_KEPT, Kc=Kd, Vc=Vd, pos_ids=pd, mass=md,
                                   ws=ws, dev_status=flag)
    torch.cuda.synchronize()
    rr = n - k
    assert flag.item() == 0 and out.shape == (B, N - rr, C) and (i32(new_len) == N - rr).all()
    if rr == 0:
        assert torch.equal(out, hd)
        return
    g_assign = i32(L.nearest_assignment(ws, B, rr))
    # a different choice must be a near-tie of the two similarities in the oracle
    for b, q in zip(*np.nonzero(g_assign != ref["assign"])):
        x = f64(hidden)[b, i0:i0 + n]
        kept = np.nonzero(rank[b] < k)[0]
        dtok = np.nonzero(rank[b] >= k)[0][q]
        cos = lambda t: float(x[kept[t]] @ x[dtok] / np.linalg.norm(x[kept[t]]) / np.linalg.norm(x[dtok]))
        a, c = cos(ref["assign"][b, q]), cos(g_assign[b, q])
        assert abs(a - c) <= 1e-4 * max(abs(a), abs(c)), "assignment differs and is not a near-tie"
    want = O.nearest_kept_merge(f64(hidden), rank, i0, n, k, mass=mass, Kc=f64(Kc) if with_kv else None,
                                Vc=f64(Vc) if with_kv else None, pos_ids=pos, assign=g_assign)
    M = N - rr
    assert_rows_close(f64(out), want["hidden"], what="merged hidden rows")
    assert torch.equal(out[:, :i0], hd[:, :i0]) and torch.equal(out[:, i0 + k:], hd[:, i0 + n:])
    assert np.array_equal(i32(pd)[:, :M], want["pos_ids"])
    if with_mass:
        assert np.array_equal(md.cpu().numpy()[:, :M], want["mass"])
    if with_kv:
        assert_rows_close(f64(Kd)[:, :, :M], want["Kc"], what="merged K rows")
        assert_rows_close(f64(Vd)[:, :, :M], want["Vc"], what="merged V rows")
        assert np.array_equal(f64(Kd)[:, :, i0 + k:M], f64(Kc)[:, :, i0 + n:])       # text rows only move


def test_nearest_kept_exact_tie_goes_to_the_lower_kept_index():
    """Two identical kept rows that one CTA meets in different column tiles and different halves of its
    accumulator (kept indices 130 and 260, 300 kept tokens, 148 CTAs so that the columns are not split over
    CTAs): a dropped row equal to them has to go to the lower index, exactly."""
    B, n, k, C = 37, 812, 300, 64
    r = np.random.default_rng(77)
    x = r.normal(size=(B, n, C)).astype(np.float32)
    x[:, 260] = x[:, 130]
    x[:, 700] = x[:, 130]                      # a dropped token that is the same row
    hidden = torch.from_numpy(x).to(torch.bfloat16)
    score = np.tile(np.linspace(1.0, 0.0, n, dtype=np.float32), (B, 1))     # the first k tokens are kept
    rank, _, _, _ = O.select_topk(score, k)
    hd, rd = hidden.cuda(), torch.from_numpy(rank).cuda()
    d = L.merge_dims(hd, rd, i0=0, k=k)
    d.merge_mode = L.W_NEAREST_KEPT
    ws = L.alloc_workspace(L.OP_MERGE_COMPACT, d, hd.device)
    flag = status_tensor()
    L.merge_compact(hd, rd, i0=0, k=k, mode=L.W_NEAREST_KEPT, ws=ws, dev_status=flag)
    torch.cuda.synchronize()
    assert flag.item() == 0
    g_assign = i32(L.nearest_assignment(ws, B, n - k))
    assert (g_assign[:, 700 - k] == 130).all()
    ref = O.nearest_kept_merge(f64(hidden), rank, 0, n, k)
    assert (ref["assign"][:, 700 - k] == 130).all()


# ------------------------------------------------------------------ library-internal cross-checks
def test_results_do_not_depend_on_programmatic_dependent_launch():
    """The same chain of calls with and without programmatic dependent launch, bit for bit (no kernel
    may touch its inputs before the kernels ahead of it have finished)."""
    from paper_2509_00419_b200 import build as Bld
    w = I.shrink(I.CFG1, n=448, T=64, C=512, planted=8)
    L.use_library(Bld.build_test())           # the build that carries the switch; the library proper has none
    lib = L.lib()

    def chain():
        hidden = I.hidden_states(w).cuda()
        pos = torch.arange(w.N, dtype=torch.int32)[None].cuda()
        Q, K, V = [t.cuda() for t in I.layer_qkv(w, 0, pos.cpu())]
        k = w.n // 3
        score, head = L.score_tokens(Q[:, w.n:], K, N=w.N, i0=0, n=w.n, q_lo=w.n, q_hi=w.N, want_head=True)
        rank, _, _ = L.select_topk(score, k)
        out, _ = L.merge_compact(hidden, rank, i0=0, k=k, Kc=K, Vc=V, pos_ids=pos)
        M = out.shape[1]
        ln = torch.full((w.B, w.Hkv), M, dtype=torch.int32, device="cuda")
        acc = torch.rand(w.B, w.Hkv, w.N, device="cuda")
        L.kv_compress(K, V, acc, ln, beta=0.9)
        q = I.normal_bf16(w.seed, "pdl/q", (w.B, w.H, 128)).cuda()
        dec = L.decode_attn(q, K, V, ln, acc_score=acc)
        torch.cuda.synchronize()
        return [score, rank, out, K, V, pos, ln, acc, dec]

    try:
        lib.lvlm_debug_set_pdl(0)
        torch.manual_seed(3)
        plain = chain()
        lib.lvlm_debug_set_pdl(1)
        torch.manual_seed(3)
        overlapped = chain()
    finally:
        L.use_library(None)
    assert not hasattr(L.lib(), "lvlm_debug_set_pdl")        # the library proper exports no switch
    for a, b in zip(plain, overlapped):
        assert torch.equal(a, b)


# ------------------------------------------------------------------ prefill attention with the scores as a by-product
ATTN_CASES = [  # B, N, H, Hkv, q_lo, i0, n, causal
    (1, 128, 2, 1, 100, 0, 90, True), (2, 300, 4, 2, 250, 7, 200, True), (1, 517, 7, 1, 400, 3, 390, True),
    (1, 260, 2, 2, 0, 0, 260, True), (2, 130, 4, 4, 64, 0, 64, False),
]


@pytest.mark.parametrize("case", ATTN_CASES)
def test_prefill_attn_with_scores(case):
    B, N, H, Hkv, q_lo, i0, n, causal = case
    r = np.random.default_rng(N + H)
    bf = lambda *s: torch.from_numpy(r.normal(size=s).astype(np.float32)).to(torch.bfloat16)
    Q, K, V = bf(B, N, H, 128), bf(B, Hkv, N + 5, 128), bf(B, Hkv, N + 5, 128)
    want = O.attention_with_scores(f64(Q), f64(K)[:, :, :N], f64(V)[:, :, :N], q_lo, N, i0, n, causal=causal)
    flag = status_tensor()
    out, lse, score, head = L.prefill_attn(Q.cuda(), K.cuda(), V.cuda(), N=N, causal=causal, window=(q_lo, N),
                                           i0=i0, n=n, want_head=True, dev_status=flag)
    torch.cuda.synchronize()
    assert flag.item() == 0
    assert_rows_close(f64(out), want["out"], what="attention output")
    assert np.allclose(lse.cpu().numpy(), want["lse"], rtol=1e-3, atol=1e-3)
    assert_scores_close(f64(score), want["score"], what="score from the attention pass")
    assert_scores_close(f64(head), want["score_head"], what="score_head from the attention pass")
    # the same scores as the stand-alone entry point gives (which pays a pass of its own for the normalisers)
    s2, h2 = L.score_tokens(Q.cuda()[:, q_lo:], K.cuda(), N=N, i0=i0, n=n, q_lo=q_lo, q_hi=N, causal=causal, want_head=True)
    assert_scores_close(f64(score), f64(s2), what="fused against stand-alone scoring")
    # attention only: no window, no workspace
    out2, lse2, none_s, _ = L.prefill_attn(Q.cuda(), K.cuda(), V.cuda(), N=N, causal=causal)
    torch.cuda.synchronize()
    assert none_s is None and torch.equal(out2, out) and torch.equal(lse2, lse)


def test_prefill_attn_is_repeatable_over_many_launches():
    """The attention kernel hands tiles between three kinds of warps through barriers and tensor memory: a race
    there shows up as one wrong CTA in some launches.  Several hundred CTAs (more than one wave), twenty-four
    launches: every launch must give the bits of the first one (whose values the full-size test compares with
    the oracle on the same shape)."""
    B, N, H, Hkv = 1, 3008, 28, 4
    g = torch.Generator(device="cuda").manual_seed(7)
    Q = torch.randn(B, N, H, 128, device="cuda", generator=g).to(torch.bfloat16)
    K = torch.randn(B, Hkv, N, 128, device="cuda", generator=g).to(torch.bfloat16)
    V = torch.randn(B, Hkv, N, 128, device="cuda", generator=g).to(torch.bfloat16)
    flag = status_tensor()
    first, lse_first, _, _ = L.prefill_attn(Q, K, V, N=N, dev_status=flag)
    first, lse_first = first.clone(), lse_first.clone()
    for it in range(24):
        out, lse, _, _ = L.prefill_attn(Q, K, V, N=N, dev_status=flag)
        assert torch.equal(out, first) and torch.equal(lse, lse_first), f"launch {it + 2} differs from the first"
    assert flag.item() == 0
