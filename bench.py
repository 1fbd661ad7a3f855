"""Benchmark of the LightVLM hot path on B200: pyramid token reduction, one-off KV-cache
compression and decode attention over the compressed cache, on seeded synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]
                    [--extras cfg1,cfg3,cfg4,cfg5|none]

Prints ONE JSON line.  A step is one pass of the whole path over one batch of the headline
workload (cfg2: the 7B-class pyramid at layers 5/9/13, then beta-threshold compression of the
caches of layers 6..27, then one decode step over all 28 layers).  Results for the other
configurations (batched prefill, long decode with periodic compression, 26B-class) ride along
under "workloads".  With N > 1 every rank runs its own replica (independent sequences, no
collective on the data path) and rank 0 reports the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch


# dram__bytes_read.sum + dram__bytes_write.sum per launch from one ncu capture of the kernel as it stands
# (set back to None whenever that kernel changes); the capture and its command are in the named file
NCU_TRAFFIC = {
    # stage 1 of cfg3: row_stream_kernel 365.4 + 108.6 MB, inplace_compact_kernel 78.5 + 27.9 MB, merge_plan_kernel
    # 0.25 MB
    ("cfg3", "lvlm_merge_compact"): {"bytes_per_launch": 580700000,
                                     "source": "profiles/row_stream_kernel_cfg3.txt + profiles/inplace_compact_kernel_cfg3.txt"
                                               " + profiles/merge_plan_kernel_cfg3.txt"},
}
DOMINANT_KERNEL = {"lvlm_decode_attn": "decode_cluster_kernel", "lvlm_score_tokens": "score_tc_kernel<0> + <1>",
                   "lvlm_merge_compact": "row_stream_kernel (with merge_plan_kernel before and inplace_compact_kernel after it)",
                   "lvlm_kv_compress": "kv_plan + inplace_compact kernels"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index=0):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
                for nm, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


class Flusher:
    """Evicts L2 (126 MB) between timed iterations: overwrites a 384 MB buffer, then reads a second
    one, so that the timed kernels neither find their data in L2 nor pay for writing back somebody
    else's dirty lines."""
    def __init__(self, device, mb=384):
        self.buf = torch.empty(mb << 20, dtype=torch.uint8, device=device)
        self.rd = torch.zeros(mb << 18, dtype=torch.int32, device=device)
        self.v = 0

    def __call__(self):
        self.v = (self.v + 1) & 0x7F
        self.buf.fill_(self.v)
        self.sink = self.rd.max()


def timed(fn, steps, warmup, flush, between=None):
    """Mean device time (ms) of ``fn`` over ``steps`` runs after ``warmup`` runs, CUDA events on
    the launching stream.  ``between`` (restoring tensors that are compacted in place) and the
    L2 flush run outside the event pairs."""
    ts = []
    for it in range(warmup + steps):
        if between is not None:
            between()
        if flush is not None:
            flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        e1.synchronize()
        if it >= warmup:
            ts.append(e0.elapsed_time(e1))
    return float(np.mean(ts)), ts


# ------------------------------------------------------------------------------------------
# prefill: pyramid reduction stages
# ------------------------------------------------------------------------------------------
def bench_prefill(w, device, steps, warmup, flush, peaks, breakdown=True):
    from paper_2509_00419_b200 import pipeline as P
    run = P.PyramidPrefill(w, device)
    g = P.capture(run.step)
    ms, _ = timed(g.replay, steps, warmup, flush, between=run.restore)
    res = {"ms_per_step": ms, "tokens_in": run.tokens_in,
           "tokens_per_s": run.tokens_in / (ms * 1e-3), "launches": run.launches, "stages": []}
    if breakdown:
        for s, st in enumerate(run.stages):
            hidden_in = run.hidden0 if s == 0 else run.stages[s - 1].hidden_out
            # every call captured in a graph of its own, so that no host time is measured
            g_sc = P.capture(lambda: st.run_score(run.Q[s], run.K[s]))
            g_se = P.capture(st.run_select)
            g_me = P.capture(lambda: st.run_merge(hidden_in, run.K[s], run.V[s], run.pos[s]))
            run.restore()
            t_sc, _ = timed(g_sc.replay, steps, warmup, flush, between=run.restore)
            t_se, _ = timed(g_se.replay, steps, warmup, flush)
            t_me, _ = timed(g_me.replay, steps, warmup, flush, between=run.restore)
            by = st.bytes_merge_hidden() + st.bytes_merge_kv()
            res["stages"].append({
                "n_in": st.n, "n_out": st.M, "score_ms": t_sc, "select_ms": t_se,
                "merge_compact_ms": t_me, "merge_compact_bytes": by, "score_flops": st.flops_score(),
                "merge_compact_gbs": by / (t_me * 1e6),
                "merge_compact_frac_hbm": by / (t_me * 1e6) / peaks["hbm_gbs"],
                "score_tflops": st.flops_score() / (t_sc * 1e9),
                "score_frac_tensor": st.flops_score() / (t_sc * 1e9) / peaks["bf16_tflops"]})
        # the similarity-merge variant (not in the paper) on stage 1: every dropped token into its most similar kept token
        from paper_2509_00419_b200 import binding as L
        st0 = run.stages[0]
        nk = P.ReduceStage(st0.B, st0.N, st0.C, st0.H, st0.Hkv, st0.cap, st0.i0, st0.n, st0.M, device,
                           mode=L.W_NEAREST_KEPT)
        nk.rank.copy_(st0.rank)
        g_nk = P.capture(lambda: nk.run_merge(run.hidden0, run.K[0], run.V[0], run.pos[0]))
        run.restore()
        t_nk, _ = timed(g_nk.replay, steps, warmup, flush, between=run.restore)
        del g_nk
        res["nearest_kept_stage1"] = {"merge_compact_ms": t_nk, "similarity_flops": nk.flops_similarity(),
                                      "tflops_over_whole_call": nk.flops_similarity() / (t_nk * 1e9),
                                      "frac_tensor_over_whole_call": nk.flops_similarity() / (t_nk * 1e9) / peaks["bf16_tflops"]}
        del nk
    return res, run


# ------------------------------------------------------------------------------------------
# selection on scores that pile up in a few values
# ------------------------------------------------------------------------------------------
def bench_select_ties(device):
    """lvlm_select_topk on one sequence of n scores: spread out, all equal, four distinct values (us, best of 8)."""
    from paper_2509_00419_b200 import binding as L
    from paper_2509_00419_b200 import pipeline as P
    res = {}
    for n in (16384, 65536):
        g = torch.Generator().manual_seed(n)
        cases = {"spread": torch.rand(1, n, generator=g) ** 4, "all_equal": torch.full((1, n), 0.25),
                 "four_values": torch.randint(0, 4, (1, n), generator=g).float() * 0.125}
        row = {}
        for name, sc in cases.items():
            sc = sc.to(device)
            rank = torch.empty(1, n, dtype=torch.int32, device=device)
            gr = P.capture(lambda: L.select_topk(sc, n // 4, want_kept=False, rank_out=rank))
            ts, _ = timed(gr.replay, 8, 3, None)
            row[name] = round(ts * 1e3, 1)
            del gr
        res[str(n)] = row
    return res


# ------------------------------------------------------------------------------------------
# the layer's attention with the scores as its by-product, against attention + stand-alone scoring
# ------------------------------------------------------------------------------------------
def bench_prefill_attn(w, device, steps, warmup, flush, peaks):
    """Stage-1 layer of ``w``: (a) lvlm_prefill_attn alone plus lvlm_score_tokens on the text window (which pays
    a pass of its own for the row normalisers), (b) lvlm_prefill_attn asked for the scores itself."""
    from paper_2509_00419_b200 import binding as L
    from paper_2509_00419_b200 import inputs as I
    from paper_2509_00419_b200 import pipeline as P
    layer = w.stages[0][0]
    pos = torch.arange(w.N, dtype=torch.int32, device=device)[None].repeat(w.B, 1)
    q, k, v = I.layer_qkv(w, layer, pos, device)
    q_lo = w.i0 + w.n
    out = torch.empty_like(q)
    lse = torch.empty(w.B, w.H, w.N, dtype=torch.float32, device=device)
    score = torch.empty(w.B, w.n, dtype=torch.float32, device=device)
    d = L.Dims(B=w.B, H=w.H, Hkv=w.Hkv, D=128, N=w.N, cap=k.shape[2], i0=w.i0, n=w.n, q_lo=q_lo, q_hi=w.N, causal=1)
    ws = L.alloc_workspace(L.OP_PREFILL_ATTN, d, device)
    qwin = q[:, q_lo:]

    def separate():
        L.prefill_attn(q, k, v, N=w.N, out=out, lse=lse)
        L.score_tokens(qwin, k, N=w.N, i0=w.i0, n=w.n, q_lo=q_lo, q_hi=w.N, score_out=score, ws=ws)

    def fused():
        L.prefill_attn(q, k, v, N=w.N, window=(q_lo, w.N), i0=w.i0, n=w.n, out=out, lse=lse, score_out=score, ws=ws)

    def attn_only():
        L.prefill_attn(q, k, v, N=w.N, out=out, lse=lse)

    # the three variants take turns inside every round, so that drift of the clock under a seconds-long run of a
    # compute-bound kernel is shared by them (the cost of the scores is a difference of two of these times)
    variants = (("attention_only", attn_only), ("attention_then_score_tokens", separate), ("fused", fused))
    graphs = {name: P.capture(fn) for name, fn in variants}
    samples = {name: [] for name, _ in variants}
    for it in range(warmup + steps):
        for name, _ in variants:
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); graphs[name].replay(); e1.record()
            e1.synchronize()
            if it >= warmup:
                samples[name].append(e0.elapsed_time(e1))
    t = {name: float(np.mean(v)) for name, v in samples.items()}
    del graphs
    flops = 4.0 * w.B * w.H * 128 * (w.N * (w.N + 1) / 2)          # causal: Q K^T and P V
    return {"ms": t, "attention_tflops": flops / (t["attention_only"] * 1e9),
            "attention_frac_tensor": flops / (t["attention_only"] * 1e9) / peaks["bf16_tflops"],
            "scores_cost_ms": {"separate": t["attention_then_score_tokens"] - t["attention_only"],
                               "fused": t["fused"] - t["attention_only"]}}


# ------------------------------------------------------------------------------------------
# the headline step: prefill pyramid + one-off compression + one decode step
# ------------------------------------------------------------------------------------------
class FullPass:
    """Phases of one step of a workload that has reduction stages, a one-off beta compression of
    the caches of layers kv_first_layer.. and a decode step over all layers."""

    def __init__(self, w, device):
        from paper_2509_00419_b200 import binding as L
        from paper_2509_00419_b200 import inputs as I
        from paper_2509_00419_b200 import pipeline as P
        self.w, self.L, self.device = w, L, device
        self.pre = P.PyramidPrefill(w, device)
        # original positions of the tokens that survive each stage (one reference pass)
        self.pre.step()
        torch.cuda.synchronize()
        stage_pos = [self.pre.pos[s][:, :st.Nout].clone() for s, st in enumerate(self.pre.stages)]
        self.pre.restore()
        stage_layers = [l for l, _ in w.stages]
        cap = ((w.N + 64 + 63) // 64) * 64
        self.dec = P.DecodeLayers(w.L, w.B, w.H, w.Hkv, cap, device)
        self.lens, self.Qwin = [], []
        pos0 = torch.arange(w.N, dtype=torch.int32, device=device)[None].repeat(w.B, 1)
        for l in range(w.L):
            s = sum(1 for sl in stage_layers if sl <= l)        # stages applied up to this layer
            pos = pos0 if s == 0 else stage_pos[s - 1]
            q, k, v = I.layer_qkv(w, l, pos, device)
            Nl = k.shape[2]
            self.dec.K[l, :, :, :Nl] = k
            self.dec.V[l, :, :, :Nl] = v
            self.dec.len[l] = Nl
            self.Qwin.append(q[:, Nl - w.T:Nl].contiguous())
            self.lens.append(Nl)
        self.K0, self.V0, self.len0 = self.dec.K.clone(), self.dec.V.clone(), self.dec.len.clone()
        first = w.kv_first_layer
        self.first = first
        self.e_lo = torch.full(((w.L - first) * w.B,), w.i0, dtype=torch.int32, device=device)
        self.e_hi = torch.tensor([self.lens[l] - w.T for l in range(first, w.L) for _ in range(w.B)],
                                 dtype=torch.int32, device=device)
        # after prefill every layer's text-window queries and keys exist, so the layers whose caches
        # have the same length are scored in one call (the layer index folds into the batch)
        self.groups = []
        l = first
        while l < w.L:
            l1 = l
            while l1 < w.L and self.lens[l1] == self.lens[l]:
                l1 += 1
            Nl, nb = self.lens[l], (l1 - l) * w.B
            d = L.Dims(B=nb, H=w.H, Hkv=w.Hkv, D=128, N=Nl, cap=cap, i0=0, n=Nl, q_lo=Nl - w.T,
                       q_hi=Nl, causal=1)
            self.groups.append({
                "l0": l, "l1": l1, "N": Nl,
                "Q": torch.cat(self.Qwin[l:l1], 0).contiguous(),
                "K": self.dec.K[l:l1].view(nb, w.Hkv, cap, 128),
                "head": self.dec.acc[l:l1].view(nb, w.Hkv, cap)[:, :, :Nl],
                "score": torch.empty(nb, Nl, dtype=torch.float32, device=device),
                "ws": L.alloc_workspace(L.OP_SCORE_TOKENS, d, device)})
            l = l1
        self.q_dec, self.k_new, self.v_new = [
            torch.stack(t) for t in zip(*[tuple(x[0] for x in I.decode_inputs(w, l, 0, 1, device))
                                          for l in range(w.L)])]

    def restore(self):
        self.pre.restore()
        self.dec.K.copy_(self.K0); self.dec.V.copy_(self.V0); self.dec.len.copy_(self.len0)
        self.dec.acc.zero_()

    def phase_reduce(self):
        self.pre.step()

    def phase_score_caches(self):
        w, L = self.w, self.L
        for g in self.groups:
            Nl = g["N"]
            L.score_tokens(g["Q"], g["K"], N=Nl, i0=0, n=Nl, q_lo=Nl - w.T, q_hi=Nl, causal=True,
                           score_out=g["score"], head_out=g["head"], ws=g["ws"])

    def phase_compress(self):
        w = self.w
        self.phase_score_caches()
        self.dec.compress(beta=w.beta, e_lo=self.e_lo, e_hi=self.e_hi, first_layer=self.first)

    def phase_decode(self):
        self.dec.decode_step(self.q_dec, self.k_new, self.v_new, accumulate=False)

    def step(self):
        self.phase_reduce()
        self.phase_compress()
        self.phase_decode()

    @property
    def launches(self):
        w = self.w
        # reduction stages; 2 scoring kernels per compressed layer + plan and compaction; one decode
        # kernel per layer
        return self.pre.launches + 2 * len(self.groups) + 2 + w.L


def bench_full(w, device, steps, warmup, flush, peaks, phases=True, fence=None):
    """``fence`` (a barrier over the ranks plus a device synchronise) brackets the timed steps."""
    from paper_2509_00419_b200 import pipeline as P
    fp = FullPass(w, device)
    g = P.capture(fp.step)
    fp.restore()
    for _ in range(warmup):                   # warm-up steps, then the ranks line up
        fp.restore(); flush(); g.replay()
    if fence is not None:
        fence()
    ms, per_step = timed(g.replay, steps, 0, flush, between=fp.restore)
    if fence is not None:
        fence()
    if not phases:
        return {"ms_per_step": ms, "launches": fp.launches, "tokens_in": fp.pre.tokens_in}, fp, per_step
    # phases, timed one by one (each from the restored state it expects)
    g_red = P.capture(fp.phase_reduce); fp.restore()
    t_red, _ = timed(g_red.replay, steps, warmup, flush, between=fp.restore)
    g_cmp = P.capture(fp.phase_compress); fp.restore()
    t_cmp, _ = timed(g_cmp.replay, steps, warmup, flush, between=fp.restore)
    g_scc = P.capture(fp.phase_score_caches); fp.restore()
    t_scc, _ = timed(g_scc.replay, steps, warmup, flush, between=fp.restore)
    fp.restore(); fp.phase_compress(); torch.cuda.synchronize()
    lens_after = fp.dec.len.clone()
    Kc, Vc = fp.dec.K.clone(), fp.dec.V.clone()

    def restore_after_compress():
        fp.dec.K.copy_(Kc); fp.dec.V.copy_(Vc); fp.dec.len.copy_(lens_after)

    g_dec = P.capture(fp.phase_decode)
    restore_after_compress()
    t_dec, _ = timed(g_dec.replay, steps, warmup, flush, between=restore_after_compress)
    kv_bytes = (int(lens_after.sum().item()) + w.L * w.B * w.Hkv) * 128 * 2 * 2
    kept = lens_after[fp.first:].float().mean().item()
    # what the compression itself has to move: K and V rows read once and the survivors written, scores
    lens_before = fp.len0[fp.first:].sum().item()
    cmp_bytes = (lens_before + int(lens_after[fp.first:].sum().item())) * 128 * 2 * 2 + lens_before * 8
    scc_flops = sum(2.0 * 2 * w.T * g["N"] * 128 * w.H * g["Q"].shape[0] for g in fp.groups)
    res = {"ms_per_step": ms, "reduce_ms": t_red, "compress_ms": t_cmp, "decode_ms": t_dec,
           "score_caches_ms": t_scc, "score_caches_flops": scc_flops, "score_caches_calls": len(fp.groups),
           "kv_compress_only_ms": max(t_cmp - t_scc, 0.0), "kv_compress_bytes": int(cmp_bytes),
           "tokens_in": fp.pre.tokens_in, "launches": fp.launches,
           "decode_kv_bytes": kv_bytes, "decode_gbs": kv_bytes / (t_dec * 1e6),
           "decode_frac_hbm": kv_bytes / (t_dec * 1e6) / peaks["hbm_gbs"],
           "mean_len_after_compress": kept, "len_before": fp.lens}
    return res, fp, per_step


# ------------------------------------------------------------------------------------------
# long decode with periodic compression (cfg4, and the decode half of cfg5)
# ------------------------------------------------------------------------------------------
def bench_decode_loop(w, device, flush, peaks, prompt_len, steps_total):
    """Runs ``steps_total`` decode steps over all layers with the periodic budgeted compression;
    every step and every compression is timed with its own event pair."""
    from paper_2509_00419_b200 import binding as L
    from paper_2509_00419_b200 import inputs as I
    from paper_2509_00419_b200 import pipeline as P
    dec = P.DecodeLayers(w.L, w.B, w.H, w.Hkv, w.cap, device)
    pos = torch.arange(prompt_len, dtype=torch.int32, device=device)[None].repeat(w.B, 1) % w.N
    T = min(w.T, prompt_len)
    for l in range(w.L):
        q, k, v = I.layer_qkv(w, l, pos, device)
        dec.K[l, :, :, :prompt_len] = k
        dec.V[l, :, :, :prompt_len] = v
        sc = torch.empty(w.B, prompt_len, dtype=torch.float32, device=device)
        L.score_tokens(q[:, prompt_len - T:].contiguous(), dec.K[l], N=prompt_len, i0=0, n=prompt_len,
                       q_lo=prompt_len - T, q_hi=prompt_len, causal=True, score_out=sc,
                       head_out=dec.acc[l][:, :, :prompt_len])
    dec.len.fill_(prompt_len)
    torch.cuda.synchronize()
    chunk = w.trigger
    snap = (dec.K.clone(), dec.V.clone(), dec.acc.clone())
    qb = torch.zeros(w.L, w.B, w.H, 128, dtype=torch.bfloat16, device=device)
    kb = torch.zeros(w.L, w.B, w.Hkv, 128, dtype=torch.bfloat16, device=device)
    vb = torch.zeros_like(kb)
    g_step = P.capture(lambda: dec.decode_step(qb, kb, vb, accumulate=True))
    g_cmp = P.capture(lambda: dec.compress(beta=1.0, budget=w.budget, recent=w.recent))
    # the captures ran the calls once: start again from the prompt state
    dec.K.copy_(snap[0]); dec.V.copy_(snap[1]); dec.acc.copy_(snap[2]); dec.len.fill_(prompt_len)
    dec.status.zero_()
    del snap
    def moved_rows(cur_len):
        """Accounting only (not on the timed path): the rows a compaction really has to move are the
        survivors behind the first evicted entry of their head."""
        ev = cur_len - w.recent
        keep_ev = w.budget - w.recent
        kept = torch.zeros(w.L, w.B, w.Hkv, cur_len, dtype=torch.bool, device=device)
        kept[..., ev:] = True
        top = dec.acc[..., :ev].topk(keep_ev, dim=-1).indices
        kept.scatter_(-1, top, True)
        first_drop = (~kept).float().argmax(dim=-1)
        return int((w.budget - first_drop).clamp(min=0).sum().item())

    t_dec, t_cmp, bytes_read, n_cmp, moved_rows_first = 0.0, 0.0, 0, 0, 0
    cur_len = prompt_len
    for c0 in range(0, steps_total, chunk):
        ns = min(chunk, steps_total - c0)
        qs, ks, vs = zip(*[I.decode_inputs(w, l, c0, ns, device) for l in range(w.L)])
        qs, ks, vs = torch.stack(qs, 1), torch.stack(ks, 1), torch.stack(vs, 1)   # [ns, L, ...]
        evs = []
        if cur_len > w.budget:
            if n_cmp == 0:
                moved_rows_first = moved_rows(cur_len)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush()                       # keeps the GPU busy while the replay is enqueued: the events then bracket device time
            e0.record(); g_cmp.replay(); e1.record()
            evs.append(("c", e0, e1))
            cur_len, n_cmp = w.budget, n_cmp + 1
        for t in range(ns):
            qb.copy_(qs[t]); kb.copy_(ks[t]); vb.copy_(vs[t])
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); g_step.replay(); e1.record()
            evs.append(("d", e0, e1))
            cur_len += 1
            bytes_read += cur_len * w.L * w.B * w.Hkv * 128 * 2 * 2
        torch.cuda.synchronize()
        for kind, e0, e1 in evs:
            if kind == "d":
                t_dec += e0.elapsed_time(e1)
            else:
                t_cmp += e0.elapsed_time(e1)
    assert int(dec.len.max().item()) == cur_len and int(dec.status.item()) == 0
    res = {"steps": steps_total, "layers": w.L, "decode_ms_total": t_dec, "compress_ms_total": t_cmp,
           "compressions": n_cmp, "ms_per_token_step": (t_dec + t_cmp) / steps_total,
           "decode_us_per_layer_step": t_dec * 1e3 / (steps_total * w.L),
           "decode_kv_bytes": bytes_read, "decode_gbs": bytes_read / (t_dec * 1e6),
           "decode_frac_hbm": bytes_read / (t_dec * 1e6) / peaks["hbm_gbs"],
           "compress_us_per_layer": (t_cmp * 1e3 / (n_cmp * w.L)) if n_cmp else None,
           "final_len": cur_len, "launches": steps_total * w.L + n_cmp * 2}
    # the same kernel with all layers folded into the batch of ONE call (not how a model decodes - its
    # layers depend on each other - but it shows what the kernel streams when a launch is large)
    nb = w.L * w.B
    ws_f = L.alloc_workspace(L.OP_DECODE_ATTN, L.kv_dims(dec.K.view(nb, w.Hkv, w.cap, 128), H=w.H), device)
    out_f = torch.empty(nb, w.H, 128, dtype=torch.bfloat16, device=device)
    fold = lambda: L.decode_attn(qb.view(nb, w.H, 128), dec.K.view(nb, w.Hkv, w.cap, 128),
                                 dec.V.view(nb, w.Hkv, w.cap, 128), dec.len.view(nb, w.Hkv),
                                 acc_score=dec.acc.view(nb, w.Hkv, w.cap), out=out_f, ws=ws_f)
    g_fold = P.capture(fold)
    t_fold, _ = timed(g_fold.replay, 10, 3, flush)
    by_fold = int(dec.len.sum().item()) * 128 * 2 * 2
    res["folded_layers_one_call"] = {"ms": t_fold, "kv_bytes": by_fold, "gbs": by_fold / (t_fold * 1e6),
                                     "frac_hbm": by_fold / (t_fold * 1e6) / peaks["hbm_gbs"]}
    if n_cmp:
        # bytes a compression has to move: every moved row of K and V read and written once, all scores
        # read (counted on the first compression; the later ones evict the same number of entries)
        by = moved_rows_first * 128 * 2 * 2 * 2 + w.L * w.B * w.Hkv * (w.budget + w.trigger) * 8
        res["compress_bytes_per_call"] = by
        res["compress_gbs"] = by * n_cmp / (t_cmp * 1e6)
        res["compress_frac_hbm"] = res["compress_gbs"] / peaks["hbm_gbs"]
        res["compress_timing"] = "one replay at each trigger of the loop, no warm-up (the first call of a shape is in there)"
    if cur_len > w.budget:
        # the same compression measured like every other call: the state the loop ends in (caches over the
        # budget) is compressed again and again, restored in between, after warm-up replays
        snap = (dec.K.clone(), dec.V.clone(), dec.acc.clone(), dec.len.clone())
        rows = moved_rows(cur_len)

        def restore():
            dec.K.copy_(snap[0]); dec.V.copy_(snap[1]); dec.acc.copy_(snap[2]); dec.len.copy_(snap[3])

        t_rep, _ = timed(g_cmp.replay, 5, 3, flush, between=restore)
        restore()
        del snap
        by = rows * 128 * 2 * 2 * 2 + w.L * w.B * w.Hkv * cur_len * 8
        res["compress_repeated"] = {"ms": t_rep, "bytes": by, "gbs": by / (t_rep * 1e6),
                                    "frac_hbm": by / (t_rep * 1e6) / peaks["hbm_gbs"], "len_before": cur_len,
                                    "what": "5 replays after 3 warm-up replays, caches restored in between"}
    return res


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------
_ORACLE_INPUTS = {}     # (workload, layer) -> generated tensors: the same every step, so drawn once


def oracle_full_pass(w):
    """The oracle on the same step as the GPU arm: all reduction stages, then per layer of
    kv_first_layer.. the text-window scores and the beta compression of the image span, then one
    decode step over all layers (CPU generation of the same tensors).  Returns (seconds, image
    tokens reduced, description); only the oracle calls are timed."""
    from oracle import lvlm_oracle as O
    from paper_2509_00419_b200 import inputs as I
    f64 = lambda t: t.to(torch.float64).numpy()
    hidden = f64(I.hidden_states(w))
    pos = np.arange(w.N, dtype=np.int32)[None].repeat(w.B, 0)
    n, N = w.n, w.N
    tokens, secs = 0, 0.0
    stage_of = {layer: M for layer, M in w.stages}
    caches = []
    for layer in range(w.L):
        key = (w.name, w.seed, layer)
        if key not in _ORACLE_INPUTS or _ORACLE_INPUTS[key][0].shape[2] != N:
            q, k, v = I.layer_qkv(w, layer, torch.from_numpy(pos))
            _ORACLE_INPUTS[key] = (f64(k), f64(v), f64(q[:, N - w.T:N]),
                                   [f64(t[0]) for t in I.decode_inputs(w, layer, 0, 1)])
        k, v, qwin, (dq, dk, dv) = _ORACLE_INPUTS[key]
        cap = N + 1
        Kc = np.zeros((w.B, w.Hkv, cap, w.D)); Vc = np.zeros_like(Kc)
        t0 = time.perf_counter()
        ln = np.full((w.B, w.Hkv), N, np.int32)
        Kc[:, :, :N], Vc[:, :, :N] = k, v
        if layer >= w.kv_first_layer:
            _, head = O.score_tokens(qwin, k, N - w.T, N, 0, N)
            o = O.kv_compress(Kc, Vc, np.pad(head, ((0, 0), (0, 0), (0, 1))), ln, beta=w.beta,
                              e_lo=np.full(w.B, w.i0), e_hi=np.full(w.B, N - w.T))
            Kc, Vc, ln = o["Kc"], o["Vc"], o["len"]
        O.decode_attn(dq, Kc, Vc, ln, k_new=dk, v_new=dv)
        if layer in stage_of:
            M = stage_of[layer]
            score, _ = O.score_tokens(qwin, k, w.i0 + n, N, w.i0, n)
            rank, _, _, _ = O.select_topk(score, M - 1)
            out = O.merge_compact(hidden, rank, w.i0, n, M - 1, Kc=k, Vc=v, pos_ids=pos)
            tokens += w.B * n
            hidden, pos = out["hidden"].astype(np.float64), out["pos_ids"]
            N, n = N - (n - M), M
        secs += time.perf_counter() - t0
    return secs, tokens, (f"one whole step of {w.name}: {len(w.stages)} reduction stages, scoring and beta compression "
                          f"of layers {w.kv_first_layer}..{w.L - 1}, one decode step over {w.L} layers, B={w.B}")


def _oracle_timed(w, passes=3):
    """Mean seconds of ``passes`` oracle passes after one warm-up pass."""
    secs, tokens, what = oracle_full_pass(w)                # warm-up: input generation, caches, page faults
    ts = []
    for _ in range(passes):
        secs, tokens, what = oracle_full_pass(w)
        ts.append(secs)
    return float(np.mean(ts)), tokens, what


def cpu_baseline(w):
    """The oracle as it stands on the host cores: once with every core the process may use (numpy's BLAS
    threads), once held to one thread."""
    cores = len(os.sched_getaffinity(0))
    secs, tokens, what = _oracle_timed(w)
    one = None
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            s1, _, _ = _oracle_timed(w, passes=2)
        one = tokens / s1
    except Exception:
        pass
    return {"value": tokens / secs, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": what + "; one warm-up pass, mean of 3", "seconds": secs,
            "value_one_thread": one}


# ------------------------------------------------------------------------------------------
def e2e_pass(w, device, steps, warmup):
    """The whole step through the public API with HOST buffers: every step copies all inputs of
    the step from pinned host memory (hidden states, the stages' Q windows, K, V and position ids, the
    caches and lengths of all layers, their text-window queries, the decode queries and new rows), runs
    the calls, and reads the results back (reduced hidden states, decode outputs, cache lengths)."""
    fp = FullPass(w, device)
    pre = fp.pre
    dev_in = [pre.hidden0] + pre.Q + pre.K + pre.V + pre.pos + [fp.dec.K, fp.dec.V, fp.dec.len] + \
             [g["Q"] for g in fp.groups] + [fp.q_dec, fp.k_new, fp.v_new]
    fp.restore()
    torch.cuda.synchronize()
    host_in = [t.cpu().pin_memory() for t in dev_in]
    last = pre.stages[-1]
    dev_out = [last.hidden_out, last.new_len, fp.dec.out, fp.dec.len]
    host_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in dev_out]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out)

    def step():
        for dt, ht in zip(dev_in, host_in):
            dt.copy_(ht, non_blocking=True)
        fp.dec.acc.zero_()
        fp.step()
        for ht, dt in zip(host_out, dev_out):
            ht.copy_(dt, non_blocking=True)

    ms, _ = timed(step, steps, warmup, None)
    return {"value": pre.tokens_in / (ms * 1e-3), "unit": "tokens/s", "ms_per_step": ms,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "what": "the whole step through the Python binding of the C ABI, inputs from pinned host memory, results read back"}


# ------------------------------------------------------------------------------------------
def run_reference(args, w):
    """--impl reference: the CPU oracle, as it stands, on the same workload and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ts, tokens, what = [], 0, ""
    for it in range(args.warmup + args.steps):
        secs, tokens, what = oracle_full_pass(w)
        if it >= args.warmup:
            ts.append(secs)
    ms = float(np.mean(ts)) * 1e3
    val = tokens / (ms * 1e-3)
    cores = len(os.sched_getaffinity(0))
    print(json.dumps({
        "impl": "reference", "metric": "reduced image tokens/s", "value": val, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": headline_config(w),
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def headline_config(w):
    return {"workload": w.name,
            "shape": "%d sequence(s) x (%d image + %d text tokens), %d channels, %d/%d query/KV heads of 128, %d layers"
                     % (w.B, w.n, w.T, w.C, w.H, w.Hkv, w.L),
            "stages": [[l, m] for l, m in w.stages], "beta": w.beta,
            "l2": "flushed between timed iterations (384 MB overwrite, then a 384 MB read)",
            "step": "reduce stages + score/compress layers %d..%d + one decode step over %d layers"
                    % (w.kv_first_layer, w.L - 1, w.L)}


def summary_table(name, ex):
    """Roofline fractions of one workload, a few numbers per entry point (HBM fraction of the bytes a call has to
    move, tensor fraction of the flops of a scoring call)."""
    row = {}
    pre = ex.get("prefill")
    if pre:
        row["merge_compact_hbm"] = [round(st["merge_compact_frac_hbm"], 3) for st in pre["stages"]]
        row["score_tensor"] = [round(st["score_frac_tensor"], 3) for st in pre["stages"]]
        row["select_us"] = [round(st["select_ms"] * 1e3, 1) for st in pre["stages"]]
        nk = pre.get("nearest_kept_stage1")
        if nk:
            row["nearest_kept_tensor"] = round(nk["frac_tensor_over_whole_call"], 3)
    dl = ex.get("decode_loop")
    if dl:
        row["decode_hbm"] = round(dl["decode_frac_hbm"], 3)
        row["decode_us_per_layer"] = round(dl["decode_us_per_layer_step"], 2)
        row["decode_hbm_all_layers_one_launch"] = round(dl["folded_layers_one_call"]["frac_hbm"], 3)
        if "compress_frac_hbm" in dl:
            row["kv_compress_hbm"] = round(dl["compress_frac_hbm"], 3)           # single replays inside the loop
        if "compress_repeated" in dl:
            row["kv_compress_hbm_warm"] = round(dl["compress_repeated"]["frac_hbm"], 3)   # after warm-up replays
    pa = ex.get("prefill_attn")
    if pa:
        row["prefill_attn_tensor"] = round(pa["attention_frac_tensor"], 3)
        row["scores_cost_us_separate_vs_fused"] = [round(pa["scores_cost_ms"]["separate"] * 1e3, 1),
                                                    round(pa["scores_cost_ms"]["fused"] * 1e3, 1)]
    return row


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--impl", default="lvlm", choices=["lvlm", "reference"])
    ap.add_argument("--extras", default="cfg1,cfg3,cfg4,cfg5,video")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the decode loop length")
    ap.add_argument("--only", default="", choices=["", "step", "prefill", "decode"],
                    help="run one piece and print its JSON: 'step' = the timed headline loop alone "
                         "(what a profiler should see), 'prefill' = per-call times of the reduction "
                         "stages, 'decode' = the decode loop with periodic compression")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "lvlm" else args.warmup

    from paper_2509_00419_b200 import inputs as I
    w = I.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not launched by torchrun: start one rank per GPU ourselves and let rank 0 print the line
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2509_00419_b200 import sharding as S
    w = S.shard_workload(w, rank, world)                     # every rank its own sequences
    from paper_2509_00419_b200 import build as Bld
    from paper_2509_00419_b200 import binding as L
    if rank == 0:
        Bld.build()
    if world > 1:
        dist.barrier()
    L.lib()
    peaks = load_peaks()
    flush = Flusher(device)
    if args.layers:
        w = I.shrink(w, L=args.layers)
    if args.only in ("prefill", "decode"):
        if args.only == "prefill":
            piece, run = bench_prefill(w, device, args.steps, args.warmup, flush, peaks)
        else:
            prompt = w.N if not w.stages else w.stages[-1][1] + w.T + w.i0
            piece = bench_decode_loop(w, device, flush, peaks, prompt,
                                      args.decode_steps or w.decode_steps)
        print(json.dumps({"only": args.only, "workload": w.name, "layers": w.L, "result": piece,
                          "peaks": peaks}))
        return

    sampler = ClockSampler(local)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    def fence():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    res, fp, per_step = bench_full(w, device, args.steps, args.warmup, flush, peaks,
                                   phases=args.only != "step", fence=fence)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if args.only == "step":
        print(json.dumps({"only": "step", "workload": w.name, "ms_per_step": res["ms_per_step"],
                          "launches_per_step": res["launches"], "clocks": clocks}))
        return
    value, ms = S.aggregate_throughput(res["tokens_in"], res["ms_per_step"], world, device)
    tokens = res["tokens_in"] * world
    # dominant call of the step: merge+compact of stage 1 (hidden, K, V rows), bytes per call
    stage_break, _ = bench_prefill(w, device, args.steps, args.warmup, flush, peaks)
    calls = []
    for s, st in enumerate(stage_break["stages"]):
        calls += [(f"stage{s + 1}.score", st["score_ms"]), (f"stage{s + 1}.select", st["select_ms"]),
                  (f"stage{s + 1}.merge_compact", st["merge_compact_ms"])]
    # the step by kind of call: time per step, launches, and the roofline that bounds the kind
    st_all = stage_break["stages"]
    n_st = len(st_all)
    kinds = {
        "lvlm_score_tokens": {
            "bound": "tensor", "unit": "TFLOP/s", "peak": peaks["bf16_tflops"],
            "ms": sum(x["score_ms"] for x in st_all) + res["score_caches_ms"],
            "work": sum(x["score_flops"] for x in st_all) + res["score_caches_flops"],
            "calls": n_st + res["score_caches_calls"], "launches": 2 * (n_st + res["score_caches_calls"])},
        "lvlm_merge_compact": {
            "bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"],
            "ms": sum(x["merge_compact_ms"] for x in st_all), "work": sum(x["merge_compact_bytes"] for x in st_all),
            "calls": n_st, "launches": 3 * n_st},
        "lvlm_kv_compress": {
            "bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"], "ms": res["kv_compress_only_ms"],
            "work": res["kv_compress_bytes"], "calls": 1, "launches": 2},
        "lvlm_decode_attn": {
            "bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"], "ms": res["decode_ms"],
            "work": res["decode_kv_bytes"], "calls": w.L, "launches": w.L},
    }
    rooflines = {}
    for name, kd in kinds.items():
        ach = kd["work"] / (kd["ms"] * (1e9 if kd["bound"] == "tensor" else 1e6)) if kd["ms"] > 0 else 0.0
        rooflines[name] = {"bound": kd["bound"], "achieved": ach, "peak": kd["peak"], "unit": kd["unit"],
                           "frac": ach / kd["peak"], "traffic": None, "ms_per_step": kd["ms"],
                           "ms_per_call": kd["ms"] / kd["calls"], "calls_per_step": kd["calls"],
                           "launches_per_step": kd["launches"],
                           "algorithmic_work_per_call": kd["work"] / kd["calls"]}
    rooflines["lvlm_select_topk"] = {"bound": "latency", "ms_per_step": sum(x["select_ms"] for x in st_all),
                                     "calls_per_step": n_st, "launches_per_step": n_st}
    # ---- the other configurations (rank 0, one GPU): they carry the launches big enough to be bandwidth-bound ----
    extras = {}
    if rank == 0 and world == 1:
        names = [x for x in args.extras.split(",") if x and x != "none"]
        for name in names:
            wx = I.WORKLOADS[name]
            try:
                ex = {}
                if wx.stages:
                    ex["prefill"], run = bench_prefill(wx, device, max(5, args.steps // 2), 3, flush, peaks)
                    del run
                    torch.cuda.empty_cache()
                    if name in ("cfg3", "cfg5"):
                        ex["prefill_attn"] = bench_prefill_attn(wx, device, 5, 3, flush, peaks)
                        torch.cuda.empty_cache()
                if wx.decode_steps > 1:
                    prompt = wx.N if not wx.stages else wx.stages[-1][1] + wx.T + wx.i0
                    nsteps = args.decode_steps or wx.decode_steps
                    ex["decode_loop"] = bench_decode_loop(wx, device, flush, peaks, prompt, nsteps)
                    torch.cuda.empty_cache()
                extras[name] = ex
            except Exception as e:          # an extra must not take the headline down
                import traceback
                extras[name] = {"error": repr(e), "trace": traceback.format_exc()[-600:]}
    # ---- the roofline entry: the dominant kernel of a launch that CAN be bandwidth-bound ------------------------
    # The headline step (cfg2, one sequence) moves 1-30 MB per launch and is latency-bound; its own dominant entry
    # point is listed under "rooflines".  The entry below is the streaming kernel of lvlm_merge_compact on stage 1
    # of cfg3 (16 sequences, about 600 MB per call), timed as the whole call: plan + streaming pass + compaction.
    roof_src = extras.get("cfg3", {}).get("prefill")
    if roof_src is None and rank == 0 and world == 1:
        roof_src, run = bench_prefill(I.WORKLOADS["cfg3"], device, max(5, args.steps // 2), 3, flush, peaks, breakdown=True)
        del run
        torch.cuda.empty_cache()
    if roof_src is not None:
        st1 = roof_src["stages"][0]
        tr = NCU_TRAFFIC.get(("cfg3", "lvlm_merge_compact"))
        roofline = {"bound": "hbm", "achieved": st1["merge_compact_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": st1["merge_compact_frac_hbm"], "traffic": tr["bytes_per_launch"] if tr else None,
                    "workload": "cfg3 stage 1 (16 x (1792 image + 96 text tokens) -> 1060, 4096 channels, K and V of 8 heads)",
                    "kernel": DOMINANT_KERNEL["lvlm_merge_compact"], "entry_point": "lvlm_merge_compact",
                    "algorithmic_bytes_per_call": st1["merge_compact_bytes"], "ms_per_call": st1["merge_compact_ms"],
                    "achieved_is": "algorithmic bytes of the call / mean duration of the whole call (3 launches) in graph replays",
                    "peak_source": peaks["source"] + (" (of measured)" if peaks["source"] == "measured" else " (of fallback)")}
        if tr:
            roofline["traffic_source"] = tr["source"]
    else:
        dominant = max(kinds, key=lambda k: kinds[k]["ms"] * kinds[k]["calls"] / kinds[k]["launches"])
        roofline = dict(rooflines[dominant], kernel=DOMINANT_KERNEL.get(dominant, dominant), entry_point=dominant,
                        workload=w.name,
                        peak_source=peaks["source"] + (" (of measured)" if peaks["source"] == "measured" else " (of fallback)"))
    summary = {w.name: {k: round(v["frac"], 3) for k, v in rooflines.items() if "frac" in v}}
    for name, ex in extras.items():
        if "error" not in ex:
            summary[name] = summary_table(name, ex)
    cfg = headline_config(w)
    out = {
        "metric": "reduced image tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": cfg,
        "roofline": roofline,
        "summary": summary,
        "phases_ms": {"reduce": res["reduce_ms"], "kv_compress": res["compress_ms"], "decode": res["decode_ms"]},
        "calls_ms": dict(calls),
        "decode": {"value": res["decode_gbs"], "unit": "GB/s", "frac_of_hbm_peak": res["decode_frac_hbm"],
                   "kv_bytes_per_step": res["decode_kv_bytes"],
                   "mean_len_after_compress": res["mean_len_after_compress"]},
        "rooflines": rooflines, "clocks": clocks, "gpu_launches": res["launches"] * args.steps,
        "peaks": peaks,
    }
    if rank == 0 and world == 1:
        out["e2e"] = e2e_pass(w, device, args.steps, args.warmup)
        out["cpu_baseline"] = cpu_baseline(w)
        # how many image entries per head the cumulative-attention threshold keeps, by beta (Section 3.2.2:
        # shallow layers keep more, deep layers fewer; here every layer has the same synthetic mass profile)
        sweep = {}
        for beta in (0.9, 0.95, 0.99, 0.995, 0.999):
            fp.restore()
            fp.phase_score_caches()
            fp.dec.compress(beta=beta, e_lo=fp.e_lo, e_hi=fp.e_hi, first_layer=fp.first)
            torch.cuda.synchronize()
            img_before = torch.tensor([fp.lens[l] - w.T - w.i0 for l in range(fp.first, w.L)], device=device).float()
            kept = fp.dec.len[fp.first:].float().mean(dim=(1, 2)) - w.T - w.i0
            sweep[str(beta)] = {"mean_kept_image_entries": float(kept.mean().item()),
                                "mean_kept_fraction": float((kept / img_before).mean().item())}
        fp.restore()
        extras["beta_sweep_" + w.name] = sweep
        extras["select_ties_us"] = bench_select_ties(device)
        out["workloads"] = extras
    elif rank == 0:
        out["e2e"] = {"value": None, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                      "what": "measured at N=1 only"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
