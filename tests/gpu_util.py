"""Helpers shared by the GPU parity tests (no arithmetic of the method lives here)."""
import numpy as np
import torch

ACT_TOL = 1e-2    # activations: max relative L2 error vs the oracle (bf16 storage, fp32 accumulation)
GRAD_TOL = 2e-2   # gradients


def rel_l2(got, want) -> float:
    """||got - want||_2 / ||want||_2 in fp64; absolute if the reference norm is ~0."""
    g = got.detach().double().cpu().numpy().ravel() if isinstance(got, torch.Tensor) else np.asarray(got, np.float64).ravel()
    w = want.detach().double().cpu().numpy().ravel() if isinstance(want, torch.Tensor) else np.asarray(want, np.float64).ravel()
    assert g.shape == w.shape, (g.shape, w.shape)
    assert np.all(np.isfinite(g)), "non-finite values in the GPU result"
    n = np.linalg.norm(w)
    return float(np.linalg.norm(g - w) / n) if n > 1e-12 else float(np.linalg.norm(g - w))


def bf16_randn(shape, gen, scale=1.0):
    return (torch.randn(shape, generator=gen, dtype=torch.float32) * scale).to(torch.bfloat16)


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().double().cpu().numpy()


def guard_alloc(shape, dtype, device="cuda", pad=256):
    """Allocates a tensor with NaN-filled guard bands on both sides; returns (tensor, check)."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * pad,), float("nan"), dtype=dtype, device=device)
    view = buf[pad:pad + n].view(*shape)

    def check():
        assert torch.isnan(buf[:pad]).all() and torch.isnan(buf[pad + n:]).all(), "write outside the output buffer"
    return view, check
