"""lvlm_decode_attn_static: the decode-attention entry point for callers that cannot allocate
device memory (a plug-in inside an engine that owns the whole memory pool, a binding that only
ever sees raw pointers, a loop that must not meet cudaMalloc's device-wide synchronisation).

It keeps its scratch in a fixed array inside the library, so the checks that matter are: it gives
what lvlm_decode_attn gives (and what the oracle gives), it still does so on a later call that finds the first call's
leftovers in the array, it allocates nothing, and it refuses problems that do not fit.

This file sorts after every other test file on purpose: a run that stops at the first failure has
then already run all the other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import lvlm_oracle as O
from paper_2509_00419_b200 import binding as L
from paper_2509_00419_b200 import build as B
from util import assert_rows_close, assert_scores_close, f64


def _case(seed, Bq, H, Hkv, cap, device):
    g = torch.Generator(device="cpu").manual_seed(seed)
    bf = lambda *s: torch.randn(*s, generator=g).to(torch.bfloat16).to(device)
    ln = torch.randint(1, cap - 1, (Bq, Hkv), generator=g, dtype=torch.int32)
    ln[0, 0] = cap - 1
    return dict(q=bf(Bq, H, 128), K=bf(Bq, Hkv, cap, 128), V=bf(Bq, Hkv, cap, 128),
                kn=bf(Bq, Hkv, 128), vn=bf(Bq, Hkv, 128), ln=ln.to(device),
                acc=torch.rand(Bq, Hkv, cap, generator=g).to(device))


@pytest.mark.gpu
def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    B.build()
    dev = torch.device("cuda", 0)
    # different problems back to back: each one finds the leftovers of the one before in the shared array.  The
    # last one has runs of keys too long for a CTA's logits to stay in shared memory, so it is the one that
    # really parks them in the array.
    for seed, (Bq, H, Hkv, cap) in enumerate([(2, 32, 8, 1152), (3, 28, 4, 300), (1, 8, 1, 8192)]):
        c = _case(seed, Bq, H, Hkv, cap, dev)
        ref = {k: v.clone() for k, v in c.items()}
        truth = O.decode_attn(f64(c["q"]), f64(c["K"]), f64(c["V"]), c["ln"].cpu().numpy(), k_new=f64(c["kn"]),
                              v_new=f64(c["vn"]), acc_score=c["acc"].cpu().numpy().copy())
        want = L.decode_attn(ref["q"], ref["K"], ref["V"], ref["ln"], k_new=ref["kn"], v_new=ref["vn"],
                             acc_score=ref["acc"])
        out = torch.empty_like(c["q"])
        flag = torch.zeros(1, dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        allocations = lambda: torch.cuda.memory_stats(dev)["allocation.all.allocated"]
        before = allocations()
        got = L.decode_attn_static(c["q"], c["K"], c["V"], c["ln"], k_new=c["kn"], v_new=c["vn"],
                                   acc_score=c["acc"], out=out, dev_status=flag)
        torch.cuda.synchronize()
        assert allocations() == before                   # torch's allocator was not asked for anything
        assert got.data_ptr() == out.data_ptr() and flag.item() == 0
        assert_rows_close(f64(got), f64(want), what=f"call {seed}: attention output")
        assert_rows_close(f64(got), truth["out"], what=f"call {seed}: attention output against the oracle")
        assert np.array_equal(c["ln"].cpu().numpy(), truth["len"])
        assert torch.equal(c["ln"], ref["ln"]) and torch.equal(c["K"], ref["K"]) and torch.equal(c["V"], ref["V"])
        for b in range(Bq):
            for g in range(Hkv):
                m = int(c["ln"][b, g])
                assert_scores_close(c["acc"][b, g, :m].cpu().numpy(), ref["acc"][b, g, :m].cpu().numpy(),
                                    what=f"call {seed}: acc_score")
                assert_scores_close(c["acc"][b, g, :m].cpu().numpy(), truth["acc_score"][b, g, :m],
                                    what=f"call {seed}: acc_score against the oracle")


@pytest.mark.gpu
def test_static_scratch_entry_rejects_what_does_not_fit():
    B.build()
    dev = torch.device("cuda", 0)
    Bq, H, Hkv, cap = 16, 32, 8, 4096               # needs 16*32*4096*4 = 8 MiB for the logits alone
    d = L.kv_dims(torch.empty(Bq, Hkv, cap, 128, dtype=torch.bfloat16, device="meta"), H=H)
    assert L.workspace_bytes(L.OP_DECODE_ATTN, d) > L.STATIC_SCRATCH_BYTES
    p = ctypes.c_void_p(0x1000)                      # never dereferenced: the call fails validation
    code = L.lib().lvlm_decode_attn_static(p, p, p, p, None, None, None, ctypes.byref(d),
                                           ctypes.c_float(0.1), p, None, None)
    assert code == L.ERR_WORKSPACE
    with torch.cuda.device(dev):
        torch.cuda.synchronize()                     # nothing was enqueued, the context is healthy
