"""Preallocated call sequences over the C-ABI kernels: one pyramid reduction stage, the one-off
KV-cache compression after prefill, and decode steps over all layers.  Host orchestration only
(allocation, argument marshalling, CUDA-graph capture); every step of the method runs in the
library's kernels.  Used by the benchmark and by the full-size parity tests.
"""
from __future__ import annotations

import math
from typing import List, Optional

import torch

from . import binding as L
from . import inputs as I


def pyramid_schedule(n: int, final_ratio: float, stages: int):
    """Image-token counts after each stage for a constant per-stage keep ratio that reaches
    ``final_ratio`` after ``stages`` reductions (Appendix A.2).  The library itself receives integers."""
    return [int(math.floor(n * final_ratio ** (s / stages) + 0.5)) for s in range(1, stages + 1)]


class ReduceStage:
    """score_tokens -> select_topk -> merge_compact for one layer (Section 3.2.1), with every
    output and workspace allocated once so that the calls can be captured in a CUDA graph."""

    LAUNCHES = 2 + 1 + 3      # score (normalisers, column sums + head reduction), select,
                              # merge_compact (plan, hidden, K/V)

    def __init__(self, B, N, C, H, Hkv, cap, i0, n, M, device, want_head=False, mode=L.W_LINEAR_RANK):
        self.B, self.N, self.C, self.H, self.Hkv, self.cap = B, N, C, H, Hkv, cap
        # M image tokens come out: with a merged token P_new, k = M - 1 tokens stay intact; in the
        # nearest-kept mode there is no extra token and k = M
        self.i0, self.n, self.M, self.mode = i0, n, M, mode
        self.k = M if mode == L.W_NEAREST_KEPT else M - 1
        self.q_lo, self.q_hi = i0 + n, N
        self.Nout = L.merged_rows(N, n, self.k, mode)
        f32, i32 = torch.float32, torch.int32
        self.score = torch.empty(B, n, dtype=f32, device=device)
        self.head = torch.empty(B, Hkv, n, dtype=f32, device=device) if want_head else None
        self.rank = torch.empty(B, n, dtype=i32, device=device)
        self.hidden_out = torch.empty(B, self.Nout, C, dtype=torch.bfloat16, device=device)
        self.new_len = torch.empty(B, dtype=i32, device=device)
        self.status = torch.zeros(1, dtype=i32, device=device)
        ds = L.Dims(B=B, H=H, Hkv=Hkv, D=128, N=N, cap=cap, i0=i0, n=n, q_lo=self.q_lo,
                    q_hi=self.q_hi, causal=1)
        dm = L.Dims(B=B, N=N, C=C, Hkv=Hkv, D=128, cap=cap, i0=i0, n=n, k=self.k, merge_mode=int(mode))
        self.ws_score = L.alloc_workspace(L.OP_SCORE_TOKENS, ds, device)
        self.ws_merge = L.alloc_workspace(L.OP_MERGE_COMPACT, dm, device)

    def run_score(self, Qwin, K):
        L.score_tokens(Qwin, K, N=self.N, i0=self.i0, n=self.n, q_lo=self.q_lo, q_hi=self.q_hi,
                       causal=True, score_out=self.score, head_out=self.head, ws=self.ws_score,
                       dev_status=self.status)

    def run_select(self):
        L.select_topk(self.score, self.k, want_kept=False, rank_out=self.rank,
                      dev_status=self.status)

    def run_merge(self, hidden, K, V, pos_ids):
        L.merge_compact(hidden, self.rank, i0=self.i0, k=self.k, mode=self.mode, Kc=K, Vc=V,
                        pos_ids=pos_ids, out=self.hidden_out, new_len=self.new_len,
                        ws=self.ws_merge, dev_status=self.status)

    def run(self, hidden, Qwin, K, V, pos_ids):
        self.run_score(Qwin, K)
        self.run_select()
        self.run_merge(hidden, K, V, pos_ids)
        return self.hidden_out

    # algorithmic traffic of one call, bytes (what the method itself has to move)
    def bytes_merge_hidden(self):
        return self.B * (self.N + self.Nout) * self.C * 2

    def bytes_merge_kv(self):
        return self.B * self.Hkv * (self.N + self.Nout) * 128 * 2 * 2

    def flops_similarity(self):
        """Nearest-kept mode: dropped x kept similarity, 2 r k C per sequence."""
        return 2.0 * (self.n - self.k) * self.k * self.C * self.B

    def flops_score(self):
        # text window rows x visible keys x D x heads, two passes (normaliser, column sums)
        T = self.q_hi - self.q_lo
        return 2.0 * 2 * T * self.N * 128 * self.H * self.B


class PyramidPrefill:
    """All reduction stages of one workload on seeded synthetic tensors.  Stage s takes the
    hidden states the previous stage produced; its layer's Q (text-window rows), K and V are
    generated for the tokens that survived (their original positions decide which keys are
    planted).  ``restore()`` puts back what the in-place compaction of K, V and the position ids
    overwrote."""

    def __init__(self, w: I.Workload, device, want_head=False):
        self.w, self.device = w, device
        self.hidden0 = I.hidden_states(w, device)
        self.stages: List[ReduceStage] = []
        self.Q, self.K, self.V, self.pos = [], [], [], []
        self.K0, self.V0, self.pos0 = [], [], []
        pos = torch.arange(w.N, dtype=torch.int32, device=device)[None].repeat(w.B, 1).contiguous()
        hidden = self.hidden0
        n, N = w.n, w.N
        for layer, M in w.stages:
            st = ReduceStage(w.B, N, w.C, w.H, w.Hkv, N, w.i0, n, M, device, want_head=want_head)
            q, k, v = I.layer_qkv(w, layer, pos[:, :N], device)
            qwin = q[:, st.q_lo:st.q_hi].contiguous()
            del q
            self.stages.append(st)
            self.Q.append(qwin); self.K.append(k); self.V.append(v); self.pos.append(pos.clone())
            self.K0.append(k.clone()); self.V0.append(v.clone()); self.pos0.append(pos.clone())
            # set-up pass: run the stage once to learn which tokens survive
            hidden = st.run(hidden, qwin, k, v, self.pos[-1])
            torch.cuda.synchronize()
            pos = self.pos[-1][:, :st.Nout].contiguous()
            n, N = M, st.Nout
        self.final_pos = pos
        self.restore()

    def restore(self):
        for a, a0 in zip(self.K + self.V + self.pos, self.K0 + self.V0 + self.pos0):
            a.copy_(a0)

    def step(self):
        hidden = self.hidden0
        for s, st in enumerate(self.stages):
            hidden = st.run(hidden, self.Q[s], self.K[s], self.V[s], self.pos[s])
        return hidden

    @property
    def launches(self):
        return ReduceStage.LAUNCHES * len(self.stages)

    @property
    def tokens_in(self):
        return sum(st.B * st.n for st in self.stages)


class DecodeLayers:
    """KV caches of several layers laid out [layer][B][Hkv][cap][D] with ragged lengths
    [layer][B][Hkv]; one decode step calls lvlm_decode_attn once per layer (layers of a real
    model run one after the other), the periodic compression calls lvlm_kv_compress once with
    the layers folded into the batch dimension."""

    def __init__(self, n_layers, B, H, Hkv, cap, device, with_acc=True):
        self.nl, self.B, self.H, self.Hkv, self.cap, self.device = n_layers, B, H, Hkv, cap, device
        bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
        self.K = torch.zeros(n_layers, B, Hkv, cap, 128, dtype=bf, device=device)
        self.V = torch.zeros(n_layers, B, Hkv, cap, 128, dtype=bf, device=device)
        self.len = torch.zeros(n_layers, B, Hkv, dtype=i32, device=device)
        self.acc = torch.zeros(n_layers, B, Hkv, cap, dtype=f32, device=device) if with_acc else None
        self.out = torch.empty(n_layers, B, H, 128, dtype=bf, device=device)
        self.status = torch.zeros(1, dtype=i32, device=device)
        dd = L.kv_dims(self.K[0], H=H)
        self.ws_dec = L.alloc_workspace(L.OP_DECODE_ATTN, dd, device)
        dk = L.kv_dims(self.K.view(n_layers * B, Hkv, cap, 128))
        self.ws_kv = L.alloc_workspace(L.OP_KV_COMPRESS, dk, device)

    def decode_step(self, q, k_new=None, v_new=None, accumulate=True, layers=None):
        """q [layer][B][H][D]; k_new, v_new [layer][B][Hkv][D] or None.  The first layer of a step may
        follow a compression of its own cache; every other layer follows the decode call of another
        layer, which does not touch this layer's cache, so its fetches may start early."""
        for i, l in enumerate(range(self.nl) if layers is None else layers):
            L.decode_attn(q[l], self.K[l], self.V[l], self.len[l],
                          k_new=None if k_new is None else k_new[l],
                          v_new=None if v_new is None else v_new[l],
                          acc_score=self.acc[l] if (accumulate and self.acc is not None) else None,
                          out=self.out[l], ws=self.ws_dec, dev_status=self.status, cache_stable=i > 0)

    def compress(self, beta=1.0, budget=0, recent=0, e_lo=None, e_hi=None, first_layer=0):
        nl = self.nl - first_layer
        shp = (nl * self.B, self.Hkv)
        L.kv_compress(self.K[first_layer:].view(*shp, self.cap, 128),
                      self.V[first_layer:].view(*shp, self.cap, 128),
                      self.acc[first_layer:].view(*shp, self.cap), self.len[first_layer:].view(*shp),
                      beta=beta, budget=budget, recent=recent, e_lo=e_lo, e_hi=e_hi, ws=self.ws_kv,
                      dev_status=self.status)

    def kv_bytes_read(self) -> int:
        """Bytes of K and V one decode step has to read at the current lengths."""
        return int(self.len.sum().item()) * 128 * 2 * 2


def capture(fn, warmup=1):
    """Runs ``fn`` eagerly ``warmup`` times, then captures it into a CUDA graph."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for _ in range(warmup):
            fn()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g
