"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers.  It holds none of the method's arithmetic
(no scoring, selection, merging, eviction or attention) and imports neither
the CUDA binding nor the CPU oracle, so both sides can be fed from it.

Every tensor is a pure function of ``(seed, name, element index)``: a 64-bit
counter hash (the splitmix64 finaliser) gives two 24-bit uniforms per element,
a Box-Muller transform turns them into one normal deviate, and the result is
rounded to bf16.  The same code runs on the CPU and on a CUDA device; the
transcendental functions may differ by an ulp between the two, so a consumer
that needs both sides to see identical bits copies the generated tensor
instead of generating it twice.

Workload shapes follow the models the paper evaluates (Section 4, Tables 2-6:
7B-, 8B- and 26B-class GQA decoders, up to 16384 image tokens) and the
attention-mass concentration it reports in Section 3.1 (a few percent of the
image tokens hold about 90 % of the image attention mass in deep layers): a
small set of "planted" image keys is pushed along a per-(batch, kv-head)
direction that every query also carries, which makes those keys dominate.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Tuple

import torch

_MASK64 = (1 << 64) - 1


def _s64(u: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant."""
    u &= _MASK64
    return u - (1 << 64) if u >= (1 << 63) else u


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)


def _lshr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lshr(x, 30)) * _C1
    x = (x ^ _lshr(x, 27)) * _C2
    return x ^ _lshr(x, 31)


def _mix64_int(x: int) -> int:
    x &= _MASK64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _MASK64
    return x ^ (x >> 31)


def stream_key(seed: int, name: str) -> int:
    """64-bit key of the tensor called ``name`` under ``seed`` (FNV-1a then mix)."""
    h = 0xCBF29CE484222325
    for ch in name.encode():
        h = ((h ^ ch) * 0x100000001B3) & _MASK64
    return _mix64_int(h ^ _mix64_int(seed + 0x632BE59BD9B4E019))


def hash_u64(seed: int, name: str, numel: int, device="cpu", start: int = 0) -> torch.Tensor:
    """int64 tensor of ``numel`` hashed counters (bit pattern = unsigned 64-bit hash)."""
    key = _s64(stream_key(seed, name))
    idx = torch.arange(start, start + numel, dtype=torch.int64, device=device)
    return _mix64(idx * _GOLDEN + key)


_CHUNK = 1 << 24


def normal_f32(seed: int, name: str, shape, device="cpu") -> torch.Tensor:
    """fp32 tensor of N(0,1) deviates, element i a function of (seed, name, i) only."""
    numel = int(math.prod(shape))
    out = torch.empty(numel, dtype=torch.float32, device=device)
    for s in range(0, numel, _CHUNK):
        m = min(_CHUNK, numel - s)
        z = hash_u64(seed, name, m, device, start=s)
        u1 = (_lshr(z, 40).to(torch.float32) + 1.0) * (1.0 / 16777216.0)      # (0, 1]
        u2 = (_lshr(z, 16) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)  # [0, 1)
        r = torch.sqrt(-2.0 * torch.log(u1))
        out[s:s + m] = r * torch.cos((2.0 * math.pi) * u2)
    return out.view(*shape)


def normal_bf16(seed: int, name: str, shape, device="cpu") -> torch.Tensor:
    return normal_f32(seed, name, shape, device).to(torch.bfloat16)


def uniform_int(seed: int, name: str, numel: int, modulo: int, device="cpu") -> torch.Tensor:
    """int64 tensor of values in [0, modulo)."""
    z = _lshr(hash_u64(seed, name, numel, device), 11)
    return z % modulo


def random_subset(seed: int, name: str, universe: int, count: int) -> torch.Tensor:
    """``count`` distinct indices of range(universe), ascending (smallest hashes win)."""
    z = _lshr(hash_u64(seed, name, universe, "cpu"), 1)
    order = torch.argsort(z, stable=True)
    return torch.sort(order[:count]).values


def unit_directions(seed: int, name: str, count: int, D: int, device="cpu") -> torch.Tensor:
    """[count, D] fp32 unit vectors."""
    g = normal_f32(seed, name, (count, D), device)
    return g / g.norm(dim=1, keepdim=True)


# --------------------------------------------------------------------------------------
# workload shapes
# --------------------------------------------------------------------------------------

@dataclass(frozen=True)
class Workload:
    """Shape of one synthetic workload.

    ``stages`` lists (layer, image tokens kept after that layer's reduction, the
    merged token included).  ``decode_*`` describe the generation phase that follows.
    """
    name: str
    seed: int
    B: int
    L: int
    C: int
    H: int
    Hkv: int
    n: int                      # image tokens
    T: int                      # text tokens after the image
    i0: int = 0                 # tokens before the image
    D: int = 128
    stages: Tuple[Tuple[int, int], ...] = ()
    planted: int = 0
    centroids: int = 0
    sigma: float = 0.3
    q_sink: float = 4.0         # every query += q_sink * u
    k_sink: float = 16.0        # planted keys += k_sink * u
    k_scale_planted: float = 1.0  # planted key rows are multiplied by this first
    beta: float = 0.995         # cumulative-attention threshold of the one-off compression
    kv_first_layer: int = 6     # first layer whose cache is compressed before generation
    decode_steps: int = 0
    budget: int = 0             # per-head cache budget of the periodic compression (0 = none)
    trigger: int = 128
    recent: int = 128
    cap: int = 0
    hh_period: int = 50         # appended keys are heavy hitters at hash % hh_period == 0

    @property
    def N(self) -> int:
        return self.i0 + self.n + self.T

    @property
    def G(self) -> int:
        return self.H // self.Hkv


# Stage counts of cfg2 come from a constant per-stage keep ratio with a 3 % final
# budget over three stages (Appendix A.2: layers 5, 9, 13): 2880 -> 895 -> 278 -> 86.
CFG1 = Workload("cfg1", seed=0, B=1, L=1, C=1024, H=8, Hkv=8, n=576, T=64,
                stages=((0, 288),), planted=16, q_sink=0.0, k_sink=0.0, k_scale_planted=4.0,
                beta=1.0, kv_first_layer=0, decode_steps=1, budget=256, recent=0, cap=1024)
CFG2 = Workload("cfg2", seed=2, B=1, L=28, C=3584, H=28, Hkv=4, n=2880, T=128,
                stages=((5, 895), (9, 278), (13, 86)), planted=64, centroids=256,
                decode_steps=1)
CFG2_ALT = Workload("cfg2_alt", seed=2, B=1, L=28, C=3584, H=28, Hkv=4, n=2880, T=128,
                    stages=((2, 1440), (8, 720), (16, 86)), planted=64, centroids=256,
                    decode_steps=1)
CFG3 = Workload("cfg3", seed=3, B=16, L=32, C=4096, H=32, Hkv=8, n=1792, T=96,
                stages=((4, 1060), (12, 627)), planted=32, centroids=256)
CFG4 = Workload("cfg4", seed=4, B=8, L=32, C=4096, H=32, Hkv=8, n=576, T=64,
                planted=12, decode_steps=4096, budget=1024, trigger=128, recent=128,
                cap=1152, beta=1.0)
CFG5 = Workload("cfg5", seed=5, B=1, L=48, C=6144, H=48, Hkv=8, n=16384, T=256,
                stages=((2, 4096), (12, 492)), planted=128, centroids=1024,
                decode_steps=2048, budget=512, trigger=128, recent=128, cap=768, beta=1.0)

# A video-length prompt (Section 4.2 evaluates video benchmarks with the same keep ratios): 64 frames of
# 512 tokens on the 7B-class shapes, 15 % kept after three stages at a constant ratio (32768 -> 17411
# -> 9251 -> 4915).
VIDEO = Workload("video", seed=7, B=1, L=28, C=3584, H=28, Hkv=4, n=32768, T=128,
                 stages=((5, 17411), (9, 9251), (13, 4915)), planted=256, centroids=1024, decode_steps=1)

WORKLOADS = {w.name: w for w in (CFG1, CFG2, CFG2_ALT, CFG3, CFG4, CFG5, VIDEO)}


def shrink(w: Workload, **kw) -> Workload:
    """A copy of ``w`` with some fields replaced (tests use reduced sizes)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(kw)
    return Workload(**d)


# --------------------------------------------------------------------------------------
# tensors
# --------------------------------------------------------------------------------------

def planted_positions(w: Workload, b: int) -> torch.Tensor:
    """Original image-token indices (0..n-1) of sequence ``b`` that are planted dominant."""
    return random_subset(w.seed, f"{w.name}/planted/b{b}", w.n, w.planted)


def planted_mask(w: Workload) -> torch.Tensor:
    """[B, N] bool over ORIGINAL positions: True at planted image tokens."""
    m = torch.zeros(w.B, w.N, dtype=torch.bool)
    for b in range(w.B):
        m[b, w.i0 + planted_positions(w, b)] = True
    return m


def hidden_states(w: Workload, device="cpu") -> torch.Tensor:
    """[B, N, C] bf16.  Image rows = centroid + sigma * noise when the workload has
    centroids (cluster structure), else N(0,1); all other rows N(0,1)."""
    x = normal_f32(w.seed, f"{w.name}/hidden", (w.B, w.N, w.C), device)
    if w.centroids > 0:
        cent = normal_f32(w.seed, f"{w.name}/centroids", (w.centroids, w.C), device)
        cid = uniform_int(w.seed, f"{w.name}/cid", w.B * w.n, w.centroids, device).view(w.B, w.n)
        img = x[:, w.i0:w.i0 + w.n, :]
        img.mul_(w.sigma).add_(cent[cid])
    return x.to(torch.bfloat16)


def layer_qkv(w: Workload, layer: int, pos_ids: torch.Tensor, device="cpu"):
    """Q [B,N',H,D], K and V [B,Hkv,N',D] (bf16) for one layer at the current sequence.

    ``pos_ids`` [B,N'] int holds the ORIGINAL position of every current row, which
    decides which keys are planted: a planted key is scaled by ``k_scale_planted`` and
    pushed by ``k_sink`` along the sink direction of its (b, kv-head); every query of
    the group carries ``q_sink`` times that direction.
    """
    B, Np = pos_ids.shape
    tag = f"{w.name}/L{layer}"
    q = normal_f32(w.seed, tag + "/q", (B, Np, w.H, w.D), device)
    k = normal_f32(w.seed, tag + "/k", (B, w.Hkv, Np, w.D), device)
    v = normal_f32(w.seed, tag + "/v", (B, w.Hkv, Np, w.D), device)
    u = unit_directions(w.seed, tag + "/sink", B * w.Hkv, w.D, device).view(B, w.Hkv, w.D)
    pm = planted_mask(w).to(device)
    is_planted = torch.gather(pm, 1, pos_ids.to(device=device, dtype=torch.int64))   # [B,N']
    pl = is_planted[:, None, :, None].to(torch.float32)
    if w.k_scale_planted != 1.0:
        k = k * (1.0 + (w.k_scale_planted - 1.0) * pl)
    if w.k_sink != 0.0:
        k = k + w.k_sink * pl * u[:, :, None, :]
    if w.q_sink != 0.0:
        uq = u.repeat_interleave(w.G, dim=1)                   # [B,H,D]
        q = q + w.q_sink * uq[:, None, :, :]
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


def decode_inputs(w: Workload, layer: int, step0: int, steps: int, device="cpu"):
    """Decode-phase tensors of ``steps`` consecutive steps starting at ``step0``:
    q [steps,B,H,D], k_new and v_new [steps,B,Hkv,D] (bf16).  Appended keys are heavy
    hitters (pushed along the sink direction) at about one position in ``hh_period``."""
    tag = f"{w.name}/L{layer}/dec"
    B = w.B
    q = torch.empty(steps, B, w.H, w.D, dtype=torch.float32, device=device)
    k = torch.empty(steps, B, w.Hkv, w.D, dtype=torch.float32, device=device)
    v = torch.empty(steps, B, w.Hkv, w.D, dtype=torch.float32, device=device)
    per_q, per_k = B * w.H * w.D, B * w.Hkv * w.D
    for name, dst, per in (("q", q, per_q), ("k", k, per_k), ("v", v, per_k)):
        numel = steps * per
        flat = dst.view(-1)
        for s in range(0, numel, _CHUNK):
            m = min(_CHUNK, numel - s)
            z = hash_u64(w.seed, tag + "/" + name, m, device, start=step0 * per + s)
            u1 = (_lshr(z, 40).to(torch.float32) + 1.0) * (1.0 / 16777216.0)
            u2 = (_lshr(z, 16) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)
            flat[s:s + m] = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    u = unit_directions(w.seed, f"{w.name}/L{layer}/sink", B * w.Hkv, w.D, device).view(B, w.Hkv, w.D)
    hh = _lshr(hash_u64(w.seed, tag + "/hh", steps * B * w.Hkv, device,
                        start=step0 * B * w.Hkv), 11) % w.hh_period == 0
    hh = hh.view(steps, B, w.Hkv, 1).to(torch.float32)
    if w.k_sink != 0.0:
        k = k + w.k_sink * hh * u[None]
    if w.q_sink != 0.0:
        q = q + w.q_sink * u.repeat_interleave(w.G, dim=1)[None]
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)
