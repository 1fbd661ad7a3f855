"""The seeded generators: determinism, distribution and structure (no method arithmetic)."""
import torch

from paper_2509_00419_b200 import inputs as I


def test_normal_is_deterministic_and_standard():
    a = I.normal_f32(7, "x", (1000, 257))
    b = I.normal_f32(7, "x", (1000, 257))
    assert torch.equal(a, b)
    assert not torch.equal(a, I.normal_f32(8, "x", (1000, 257)))
    assert not torch.equal(a, I.normal_f32(7, "y", (1000, 257)))
    assert abs(a.mean().item()) < 0.01 and abs(a.std().item() - 1.0) < 0.01
    # element i depends on (seed, name, i) only: a prefix of a longer tensor is the same
    c = I.normal_f32(7, "x", (2000 * 257,))
    assert torch.equal(c[:1000 * 257], a.view(-1))


def test_workload_structure():
    w = I.shrink(I.CFG2, n=96, T=16, C=64, planted=5, centroids=8)
    h = I.hidden_states(w)
    assert h.shape == (1, 112, 64) and h.dtype == torch.bfloat16
    pm = I.planted_mask(w)
    assert pm.sum().item() == 5 and not pm[:, w.n:].any()
    pos = torch.arange(w.N)[None]
    q, k, v = I.layer_qkv(w, 5, pos)
    assert q.shape == (1, 112, 28, 128) and k.shape == (1, 4, 112, 128) and v.shape == k.shape
    kn = k.float().norm(dim=-1)[0, 0]
    assert kn[pm[0]].min() > kn[~pm[0]].max()          # planted keys stand out
    qd, kd, vd = I.decode_inputs(w, 3, 10, 4)
    q2, _, _ = I.decode_inputs(w, 3, 12, 2)
    assert torch.equal(qd[2:], q2)                       # steps are addressable individually
    assert kd.shape == (4, 1, 4, 128)


def test_config_table_matches_the_stated_shapes():
    assert (I.CFG1.n, I.CFG1.T, I.CFG1.C, I.CFG1.H, I.CFG1.Hkv) == (576, 64, 1024, 8, 8)
    assert (I.CFG2.n, I.CFG2.T, I.CFG2.C, I.CFG2.H, I.CFG2.Hkv, I.CFG2.L) == (2880, 128, 3584, 28, 4, 28)
    assert [m for _, m in I.CFG2.stages] == [895, 278, 86] and [l for l, _ in I.CFG2.stages] == [5, 9, 13]
    assert (I.CFG3.B, I.CFG3.n, I.CFG3.T, I.CFG3.C) == (16, 1792, 96, 4096)
    assert (I.CFG4.B, I.CFG4.budget, I.CFG4.cap, I.CFG4.decode_steps) == (8, 1024, 1152, 4096)
    assert (I.CFG5.n, I.CFG5.T, I.CFG5.C, I.CFG5.H) == (16384, 256, 6144, 48)
