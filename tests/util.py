"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def i32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().astype(np.int32)


def bf16_cuda(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).cuda()


def assert_rows_close(got: np.ndarray, want: np.ndarray, rtol=1e-2, atol=1e-3, what=""):
    """bf16 rows / attention outputs: |got - want| <= atol + rtol * |want| element-wise."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    bound = atol + rtol * np.abs(want)
    bad = err > bound
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} elements off, worst {err.max():.3e}"


def assert_scores_close(got, want, rtol=1e-3, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    bound = rtol * np.abs(want) + 1e-30
    bad = err > bound
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} scores off, worst rel " \
                          f"{(err / (np.abs(want) + 1e-30)).max():.3e}"
