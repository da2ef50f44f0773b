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


# Per-element bounds, beside the norm: |gpu - oracle| <= atol_rms * rms(oracle) + rtol * |oracle|.
# A bf16 store rounds to 2^-9 relative (half an ulp), so rtol = 2^-7 leaves room for two roundings on
# the way (an intermediate stored as bf16, then the output).  The absolute term scales with the
# tensor's root-mean-square value: an output element is a sum of many products whose operands carry
# those roundings, so its error is set by the size of the terms, not by the size of the (possibly
# cancelled) sum.  A tensor that passes the norm test at e = 3e-3 with Gaussian-like errors has its
# worst of 1e8 elements near 6 e rms = 0.02 rms; a tile of wrong values is off by about rms.
ELEM_ACT = dict(atol_rms=0.04, rtol=2.0 ** -7)      # activations
ELEM_GRAD = dict(atol_rms=0.08, rtol=2.0 ** -6)     # gradients (two more bf16 hand-offs on the way)
ELEM_F32 = dict(atol_rms=2e-4, rtol=2e-4)           # fp32 statistics (mean, 1/sigma, lse)


def elem_check(got, want, name="", atol_rms=0.04, rtol=2.0 ** -7):
    """Asserts the per-element bound and returns the worst ratio |diff| / bound (<= 1 passes).
    On failure the message names the worst element's flat index, both values and the bound."""
    g = got.detach().double().cpu().numpy().ravel() if isinstance(got, torch.Tensor) else np.asarray(got, np.float64).ravel()
    w = want.detach().double().cpu().numpy().ravel() if isinstance(want, torch.Tensor) else np.asarray(want, np.float64).ravel()
    assert g.shape == w.shape, (name, g.shape, w.shape)
    assert np.all(np.isfinite(g)), f"{name}: non-finite values in the GPU result"
    rms = float(np.sqrt(np.mean(w * w)))
    bound = atol_rms * rms + rtol * np.abs(w)
    if rms == 0.0:
        bound = bound + 1e-30
    ratio = np.abs(g - w) / bound
    i = int(np.argmax(ratio))
    worst = float(ratio[i])
    assert worst <= 1.0, (f"{name}: element {i} of {g.size}: gpu {g[i]!r} vs oracle {w[i]!r}, |diff| {abs(g[i] - w[i]):.3e} "
                          f"> bound {bound[i]:.3e} (rms {rms:.3e}, atol_rms {atol_rms}, rtol {rtol}); "
                          f"{int((ratio > 1.0).sum())} elements out of bound")
    return worst


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


def dims_of(w):
    """oracle.Dims for an inputs.Workload."""
    from oracle import Dims
    return Dims(w.batch, w.seq_len, w.d_model, w.n_heads, w.head_dim, w.d_ff)


def make_layer(pw, w, act=0, flags=0):
    return pw.Layer(w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch, act=act, flags=flags)


def zeros_like_params(w, device="cuda"):
    return [torch.zeros(s, dtype=torch.float32, device=device) for s in w.param_shapes()]


def run_layer_gpu(pw, layer, params_dev, x_dev, dy_dev, save_ctx=True, grads=None, accumulate=False):
    """One forward + backward through the C ABI.  Returns dict(y, dx, grads, ctx, scratch)."""
    T, d = layer.T, layer.d
    y = torch.empty((T, d), dtype=torch.bfloat16, device="cuda")
    dx = torch.empty_like(y)
    ctx = torch.empty(layer.ctx_bytes, dtype=torch.uint8, device="cuda") if save_ctx else None
    scratch = torch.empty(layer.scratch_bytes, dtype=torch.uint8, device="cuda")
    if grads is None:
        grads = [torch.full(p.shape, float("nan"), dtype=torch.float32, device="cuda") for p in params_dev]
    layer.fwd(params_dev, x_dev, y, ctx, scratch)
    layer.bwd(params_dev, x_dev, dy_dev, dx, grads, accumulate, ctx, scratch)
    torch.cuda.synchronize()
    code, site = layer.status()
    assert code == 0, f"device status {code} at site {site}"
    return dict(y=y, dx=dx, grads=grads, ctx=ctx, scratch=scratch)
