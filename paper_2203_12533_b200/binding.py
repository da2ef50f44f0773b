"""ctypes binding over the C-ABI library ``libpw.so`` (see ``include/pw.h``).

Argument marshalling only: every step of the layer runs in the library's CUDA
kernels.  torch is used for device memory (``tensor.data_ptr()``) and streams.
There is no fallback: if the library is missing or the device is not sm_100,
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpw.so")

PW_OK = 0
STATUS_NAMES = {0: "PW_OK", 1: "PW_ERR_INVALID_ARG", 2: "PW_ERR_UNSUPPORTED_SHAPE", 3: "PW_ERR_WORKSPACE_TOO_SMALL",
                4: "PW_ERR_CUDA", 5: "PW_ERR_DEVICE_UNSUPPORTED", 6: "PW_ERR_TIMEOUT", 7: "PW_ERR_INTERNAL"}
ACT_GELU_ERF, ACT_GELU_TANH = 0, 1
FLAG_LEAN_CTX = 1
FLAG_WHOLE_LAYER = 2
GEMM_TN, GEMM_NN, GEMM_NT = 0, 1, 2
EPI_NONE, EPI_BIAS, EPI_BIAS_RESID, EPI_BIAS_GELU, EPI_DGELU, EPI_F32 = range(6)
DISPATCH_OPBYOP, DISPATCH_ASYNC, DISPATCH_GRAPH = 0, 1, 2
SCHEDULE_GPIPE, SCHEDULE_PER_MICROBATCH = 0, 1
CTX_NAMES = ("h1", "qkv", "o", "x1", "h2", "u", "a", "lse", "mu1", "r1", "mu2", "r2")
PARAM_NAMES = ("ln1_gamma", "ln1_beta", "w_qkv", "b_qkv", "w_o", "b_o",
               "ln2_gamma", "ln2_beta", "w_fc1", "b_fc1", "w_fc2", "b_fc2")

EXPORTS = (
    "pw_version", "pw_status_string", "pw_last_error",
    "pw_layer_create", "pw_layer_destroy", "pw_layer_workspace_bytes", "pw_layer_ctx_offset",
    "pw_layer_fwd", "pw_layer_bwd", "pw_layer_status",
    "pw_layer_profile_begin", "pw_layer_profile_end", "pw_layer_launch_count",
    "pw_stage_create", "pw_stage_destroy", "pw_stage_workspace_bytes", "pw_stage_run_chain", "pw_stage_status",
    "pw_stage_profile_begin", "pw_stage_profile_end", "pw_stage_launch_count",
    "pw_op_layernorm_fwd", "pw_op_layernorm_bwd_scratch_bytes", "pw_op_layernorm_bwd",
    "pw_op_colsum_scratch_bytes", "pw_op_colsum", "pw_op_colsum_noalloc", "pw_op_gemm", "pw_op_gemm_rowdot",
    "pw_op_attention_fwd", "pw_op_attention_bwd", "pw_op_status",
    "pw_lm_workspace_bytes", "pw_lm_step",
    "pw_op_embedding_fwd", "pw_op_embedding_bwd_scratch_bytes", "pw_op_embedding_bwd", "pw_op_softmax_xent",
    "pw_set_tuning", "pw_get_tuning", "pw_set_log", "pw_op_status_reset", "pw_op_selftest_wait_timeout", "pw_op_affine_f32", "pw_sgd_apply",
    "pw_layer_set_side_stream", "pw_stage_set_side_stream", "pw_dp_slice", "pw_dp_reduce_apply", "pw_shared_alloc", "pw_shared_free", "pw_shared_open", "pw_shared_close",
)


class PwError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class LayerConfig(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("d_model", ctypes.c_int32), ("n_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("seq_len", ctypes.c_int32),
                ("batch", ctypes.c_int32), ("act", ctypes.c_int32), ("ln_eps", ctypes.c_float),
                ("causal", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class IpcHandle(ctypes.Structure):
    _fields_ = [("bytes", ctypes.c_ubyte * 64)]


DP_MAX_WORLD = 8
APPLY_ITEMS_PER_LAUNCH = 64      # tensors one launch of the gradient apply serves


class ApplyItem(ctypes.Structure):
    _fields_ = [("param", ctypes.c_void_p), ("master", ctypes.c_void_p), ("grad", ctypes.c_void_p),
                ("n", ctypes.c_int64)]


KERNEL_CLASSES = ("gemm_tn", "gemm_nn", "gemm_nt", "attn_fwd", "attn_bwd", "ln_fwd", "ln_bwd", "colsum", "xent", "embed",
                  "gelu", "whole_layer", "reduce")


class Profile(ctypes.Structure):
    _fields_ = [("launches", ctypes.c_uint64 * 13), ("ms", ctypes.c_double * 13), ("flops", ctypes.c_double * 13),
                ("bytes", ctypes.c_double * 13)]

    def as_dict(self):
        return {n: dict(launches=int(self.launches[i]), ms=float(self.ms[i]), flops=float(self.flops[i]),
                        bytes=float(self.bytes[i])) for i, n in enumerate(KERNEL_CLASSES)}


class _Ptr3(ctypes.Structure):
    """pw_lm_params_t / pw_lm_grads_t: embedding table, final LayerNorm gamma, beta."""
    _fields_ = [("embedding", ctypes.c_void_p), ("lnf_gamma", ctypes.c_void_p), ("lnf_beta", ctypes.c_void_p)]


class _Ptr12(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in PARAM_NAMES]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libpw.so (built by ``paper_2203_12533_b200.build``); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2203_12533_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(_LIB_PATH)
        L.pw_version.restype = ctypes.c_int
        L.pw_status_string.restype = ctypes.c_char_p
        L.pw_status_string.argtypes = [ctypes.c_int]
        L.pw_last_error.restype = ctypes.c_char_p
        L.pw_op_layernorm_bwd_scratch_bytes.restype = ctypes.c_size_t
        L.pw_op_layernorm_bwd_scratch_bytes.argtypes = [ctypes.c_int, ctypes.c_int]
        L.pw_op_colsum_scratch_bytes.restype = ctypes.c_size_t
        L.pw_op_colsum_scratch_bytes.argtypes = [ctypes.c_int, ctypes.c_int]
        vp, ci = ctypes.c_void_p, ctypes.c_int
        L.pw_layer_create.argtypes = [ctypes.POINTER(LayerConfig), ctypes.POINTER(vp)]
        L.pw_layer_destroy.argtypes = [vp]
        L.pw_layer_destroy.restype = None
        L.pw_layer_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
        L.pw_layer_ctx_offset.argtypes = [vp, ci, ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
        L.pw_layer_fwd.argtypes = [vp, ctypes.POINTER(_Ptr12), vp, vp, vp, vp, vp]
        L.pw_layer_bwd.argtypes = [vp, ctypes.POINTER(_Ptr12), vp, vp, vp, ctypes.POINTER(_Ptr12), ci, vp, vp, vp]
        L.pw_layer_status.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.pw_layer_profile_begin.argtypes = [vp]
        L.pw_layer_profile_end.argtypes = [vp, ctypes.POINTER(Profile)]
        L.pw_layer_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64)]
        L.pw_stage_profile_begin.argtypes = [vp]
        L.pw_stage_profile_end.argtypes = [vp, ctypes.POINTER(Profile)]
        L.pw_stage_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64)]
        L.pw_stage_create.argtypes = [ctypes.POINTER(LayerConfig), ci, ctypes.POINTER(vp)]
        L.pw_stage_destroy.argtypes = [vp]
        L.pw_stage_destroy.restype = None
        L.pw_stage_workspace_bytes.argtypes = [vp, ci, ci, ci, ctypes.POINTER(ctypes.c_size_t)]
        L.pw_stage_run_chain.argtypes = [vp, ctypes.POINTER(_Ptr12), ctypes.POINTER(_Ptr12), ctypes.POINTER(vp),
                                         ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), ci, ci, ci, ci,
                                         vp, ctypes.c_size_t, vp]
        L.pw_stage_status.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.pw_op_layernorm_fwd.argtypes = [vp, vp, vp, ci, ci, ctypes.c_float, vp, vp, vp, vp]
        L.pw_op_layernorm_bwd.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, vp, vp, vp, vp, vp, ci, vp, vp]
        L.pw_op_colsum.argtypes = [vp, ci, ci, ci, vp, ci, vp, vp]
        L.pw_op_colsum_noalloc.argtypes = [vp, ci, ci, ci, vp, ci, vp]
        L.pw_op_gemm.argtypes = [ci, ci, ci, ci, ci, ci, vp, ci, vp, ci, vp, ci, vp, vp, ci, vp, ci, vp]
        L.pw_op_gemm_rowdot.argtypes = [ci, ci, ci, vp, ci, vp, ci, vp, ci, vp, ci, ci, ci, vp, vp]
        L.pw_op_attention_fwd.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp]
        L.pw_op_attention_bwd.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, vp]
        L.pw_op_status.argtypes = [ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.pw_lm_workspace_bytes.argtypes = [vp, ci, ci, ctypes.POINTER(ctypes.c_size_t)]
        L.pw_lm_step.argtypes = [vp, ctypes.POINTER(_Ptr12), ctypes.POINTER(_Ptr12), ctypes.POINTER(_Ptr3),
                                 ctypes.POINTER(_Ptr3), vp, vp, vp, ci, ci, vp, ctypes.c_size_t, vp]
        L.pw_op_embedding_fwd.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        L.pw_op_embedding_bwd_scratch_bytes.restype = ctypes.c_size_t
        L.pw_op_embedding_bwd_scratch_bytes.argtypes = [ci, ci]
        L.pw_op_embedding_bwd.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp]
        L.pw_op_softmax_xent.argtypes = [vp, ci, vp, ci, ci, ctypes.c_float, vp, vp, vp]
        L.pw_op_selftest_wait_timeout.argtypes = [ctypes.c_uint64, ctypes.POINTER(ci), vp]
        L.pw_op_affine_f32.argtypes = [vp, ctypes.c_longlong, ctypes.c_float, ctypes.c_float, vp, vp]
        L.pw_layer_set_side_stream.argtypes = [vp, ci]
        L.pw_stage_set_side_stream.argtypes = [vp, ci]
        L.pw_dp_slice.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int64),
                                  ctypes.POINTER(ctypes.c_int64)]
        L.pw_dp_reduce_apply.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, ctypes.c_int64,
                                         ctypes.c_float, ctypes.c_float, ctypes.c_int, vp]
        L.pw_shared_alloc.argtypes = [ctypes.c_size_t, ctypes.POINTER(vp), ctypes.POINTER(IpcHandle)]
        L.pw_shared_free.argtypes = [vp]
        L.pw_shared_open.argtypes = [ctypes.POINTER(IpcHandle), ctypes.POINTER(vp)]
        L.pw_shared_close.argtypes = [vp]
        L.pw_sgd_apply.argtypes = [ctypes.POINTER(ApplyItem), ctypes.c_int, ctypes.c_float, ctypes.c_float,
                                   ctypes.c_int, vp]
        _lib = L
    return _lib


def _check(status: int):
    if status != PW_OK:
        raise PwError(status, lib().pw_last_error().decode())


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _p(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda, "device tensors must be CUDA tensors"
    return t.data_ptr()


def _ptr12(tensors: Sequence) -> _Ptr12:
    assert len(tensors) == 12
    s = _Ptr12()
    for n, t in zip(PARAM_NAMES, tensors):
        setattr(s, n, _p(t))
    return s


def make_config(d_model, n_heads, head_dim, d_ff, seq_len, batch, act=ACT_GELU_ERF, ln_eps=1e-5, causal=1, flags=0):
    return LayerConfig(ctypes.sizeof(LayerConfig), d_model, n_heads, head_dim, d_ff, seq_len, batch, act, ln_eps,
                       causal, flags)


class Layer:
    """One pre-LN causal decoder layer with static shapes (pw_layer_*)."""

    def __init__(self, d_model, n_heads, head_dim, d_ff, seq_len, batch, act=ACT_GELU_ERF, ln_eps=1e-5, causal=1, flags=0):
        self.cfg = make_config(d_model, n_heads, head_dim, d_ff, seq_len, batch, act, ln_eps, causal, flags)
        self._h = ctypes.c_void_p()
        _check(lib().pw_layer_create(ctypes.byref(self.cfg), ctypes.byref(self._h)))
        a, b = ctypes.c_size_t(), ctypes.c_size_t()
        _check(lib().pw_layer_workspace_bytes(self._h, ctypes.byref(a), ctypes.byref(b)))
        self.ctx_bytes, self.scratch_bytes = a.value, b.value
        self.T, self.d, self.F = batch * seq_len, d_model, d_ff
        self.B, self.S, self.H, self.dh = batch, seq_len, n_heads, head_dim

    def close(self):
        if self._h:
            lib().pw_layer_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def ctx_view(self, ctx: torch.Tensor, name: str) -> torch.Tensor:
        """A typed view of one saved tensor inside a ctx (or ctx-shaped scratch) byte buffer."""
        i = CTX_NAMES.index(name)
        off, nb = ctypes.c_size_t(), ctypes.c_size_t()
        _check(lib().pw_layer_ctx_offset(self._h, i, ctypes.byref(off), ctypes.byref(nb)))
        if nb.value == 0:
            raise KeyError(f"{name} is not kept in this layer's ctx (lean save set)")
        raw = ctx.view(torch.uint8)[off.value:off.value + nb.value]
        T, d, F = self.T, self.d, self.F
        if name in ("h1", "o", "x1", "h2"):
            return raw.view(torch.bfloat16).view(T, d)
        if name == "qkv":
            return raw.view(torch.bfloat16).view(T, 3 * d)
        if name in ("u", "a"):
            return raw.view(torch.bfloat16).view(T, F)
        if name == "lse":
            return raw.view(torch.float32).view(self.B, self.H, self.S)
        return raw.view(torch.float32).view(T)

    def fwd(self, params, x, y, ctx, scratch, stream=None):
        _check(lib().pw_layer_fwd(self._h, ctypes.byref(_ptr12(params)), _p(x), _p(y), _p(ctx), _p(scratch),
                                  _stream(stream)))

    def bwd(self, params, x, dy, dx, grads, accumulate, ctx, scratch, stream=None):
        _check(lib().pw_layer_bwd(self._h, ctypes.byref(_ptr12(params)), _p(x), _p(dy), _p(dx),
                                  ctypes.byref(_ptr12(grads)), int(accumulate), _p(ctx), _p(scratch),
                                  _stream(stream)))

    def set_side_stream(self, enabled: bool):
        _check(lib().pw_layer_set_side_stream(self._h, int(bool(enabled))))

    def status(self):
        c, s = ctypes.c_int(), ctypes.c_int()
        _check(lib().pw_layer_status(self._h, ctypes.byref(c), ctypes.byref(s)))
        return c.value, s.value

    def profile_begin(self):
        _check(lib().pw_layer_profile_begin(self._h))

    def profile_end(self) -> dict:
        p = Profile()
        _check(lib().pw_layer_profile_end(self._h, ctypes.byref(p)))
        return p.as_dict()

    def launch_count(self) -> int:
        n = ctypes.c_uint64()
        _check(lib().pw_layer_launch_count(self._h, ctypes.byref(n)))
        return n.value


class Stage:
    """A stack of identical-shape layers run over M micro-batches (pw_stage_*)."""

    def __init__(self, n_layers, d_model, n_heads, head_dim, d_ff, seq_len, batch, act=ACT_GELU_ERF, ln_eps=1e-5, flags=0):
        self.cfg = make_config(d_model, n_heads, head_dim, d_ff, seq_len, batch, act, ln_eps, 1, flags)
        self.n_layers = n_layers
        self._h = ctypes.c_void_p()
        _check(lib().pw_stage_create(ctypes.byref(self.cfg), n_layers, ctypes.byref(self._h)))

    def close(self):
        if self._h:
            lib().pw_stage_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_bytes(self, n_microbatches, schedule=SCHEDULE_GPIPE, recompute=True) -> int:
        n = ctypes.c_size_t()
        _check(lib().pw_stage_workspace_bytes(self._h, n_microbatches, schedule, int(recompute), ctypes.byref(n)))
        return n.value

    def run_chain(self, params, grads, xs, dys, ys, dxs, workspace, dispatch=DISPATCH_ASYNC,
                  schedule=SCHEDULE_GPIPE, recompute=True, stream=None, workspace_bytes=None):
        L, M = self.n_layers, len(xs)
        assert len(params) == L and len(grads) == L
        P = (_Ptr12 * L)(*[_ptr12(p) for p in params])
        G = (_Ptr12 * L)(*[_ptr12(g) for g in grads])
        arr = lambda ts: (ctypes.c_void_p * M)(*[_p(t) for t in ts])
        nbytes = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
        _check(lib().pw_stage_run_chain(self._h, P, G, arr(xs), arr(dys), arr(ys), arr(dxs), M, dispatch, schedule,
                                        int(recompute), _p(workspace), nbytes, _stream(stream)))

    def lm_workspace_bytes(self, vocab, recompute=False) -> int:
        n = ctypes.c_size_t()
        _check(lib().pw_lm_workspace_bytes(self._h, vocab, int(recompute), ctypes.byref(n)))
        return n.value

    def lm_step(self, params, grads, lm_params, lm_grads, ids, labels, loss, vocab, workspace, recompute=False,
                stream=None, workspace_bytes=None):
        """One training step of the small LM (pw_lm_step).  lm_params = (E, lnf_gamma, lnf_beta) bf16,
        lm_grads = (dE, dlnf_gamma, dlnf_beta) fp32, ids / labels int32 [B,S], loss fp32 [1]."""
        L = self.n_layers
        assert len(params) == L and len(grads) == L
        P = (_Ptr12 * L)(*[_ptr12(p) for p in params])
        G = (_Ptr12 * L)(*[_ptr12(g) for g in grads])
        lp = _Ptr3(*[_p(t) for t in lm_params])
        lg = _Ptr3(*[_p(t) for t in lm_grads])
        nbytes = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
        _check(lib().pw_lm_step(self._h, P, G, ctypes.byref(lp), ctypes.byref(lg), _p(ids), _p(labels), _p(loss), vocab,
                                int(recompute), _p(workspace), nbytes, _stream(stream)))

    def set_side_stream(self, enabled: bool):
        _check(lib().pw_stage_set_side_stream(self._h, int(bool(enabled))))

    def status(self):
        c, s = ctypes.c_int(), ctypes.c_int()
        _check(lib().pw_stage_status(self._h, ctypes.byref(c), ctypes.byref(s)))
        return c.value, s.value

    def profile_begin(self):
        _check(lib().pw_stage_profile_begin(self._h))

    def profile_end(self) -> dict:
        p = Profile()
        _check(lib().pw_stage_profile_end(self._h, ctypes.byref(p)))
        return p.as_dict()

    def launch_count(self) -> int:
        n = ctypes.c_uint64()
        _check(lib().pw_stage_launch_count(self._h, ctypes.byref(n)))
        return n.value


# ---- single steps ----
def op_layernorm_fwd(x, gamma, beta, eps, h, mu, rstd, stream=None):
    T, d = x.shape
    _check(lib().pw_op_layernorm_fwd(_p(x), _p(gamma), _p(beta), T, d, eps, _p(h), _p(mu), _p(rstd), _stream(stream)))


def op_layernorm_bwd_scratch_bytes(T, d) -> int:
    return lib().pw_op_layernorm_bwd_scratch_bytes(T, d)


def op_layernorm_bwd(dh, x, mu, rstd, gamma, resid, dx, dgamma, dbeta, db_resid, db_dx, accumulate, partials,
                     stream=None):
    T, d = x.shape
    _check(lib().pw_op_layernorm_bwd(_p(dh), _p(x), _p(mu), _p(rstd), _p(gamma), _p(resid), T, d, _p(dx), _p(dgamma),
                                     _p(dbeta), _p(db_resid), _p(db_dx), int(accumulate), _p(partials),
                                     _stream(stream)))


def op_embedding_fwd(ids, E, x0, stream=None):
    V, d = E.shape
    _check(lib().pw_op_embedding_fwd(_p(ids), _p(E), ids.numel(), d, V, _p(x0), _stream(stream)))


def op_embedding_bwd_scratch_bytes(T, V) -> int:
    return lib().pw_op_embedding_bwd_scratch_bytes(T, V)


def op_embedding_bwd(ids, dx0, dE, scratch, stream=None):
    V, d = dE.shape
    _check(lib().pw_op_embedding_bwd(_p(ids), _p(dx0), ids.numel(), d, V, _p(dE), _p(scratch), _stream(stream)))


def op_softmax_xent(logits, labels, grad_scale, lse, loss_rows, stream=None):
    T, V = logits.shape
    _check(lib().pw_op_softmax_xent(_p(logits), logits.stride(0), _p(labels), T, V, grad_scale, _p(lse), _p(loss_rows),
                                    _stream(stream)))


def op_colsum_scratch_bytes(T, N) -> int:
    return lib().pw_op_colsum_scratch_bytes(T, N)


def op_colsum(inp, out, accumulate, partials, stream=None):
    T, N = inp.shape
    _check(lib().pw_op_colsum(_p(inp), T, N, inp.stride(0), _p(out), int(accumulate), _p(partials), _stream(stream)))


def op_colsum_noalloc(inp, out, accumulate, stream=None):
    """Column sums of a bf16 [T, N] tensor into fp32 [N] without any device allocation.

    For callers that may not allocate when they run (memory pools own all of HBM, host callbacks,
    plugins without an allocator): the partial sums live in a 1 MiB array inside libpw.so, shared
    by every call on the device, so overlapping calls must be serialised.  N <= 262144.
    """
    T, N = inp.shape
    _check(lib().pw_op_colsum_noalloc(_p(inp), T, N, inp.stride(0), _p(out), int(accumulate), _stream(stream)))


def op_gemm(layout, epilogue, M, N, K, A, lda, B, ldb, C, ldc, bias=None, aux_in=None, ld_aux=0, aux_out=None,
            accumulate=False, act=ACT_GELU_ERF, stream=None):
    _check(lib().pw_op_gemm(layout, epilogue, act, M, N, K, _p(A), lda, _p(B), ldb, _p(C), ldc, _p(bias), _p(aux_in),
                            ld_aux, _p(aux_out), int(accumulate), _stream(stream)))


def op_gemm_rowdot(M, N, K, A, lda, B, ldb, C, ldc, other, ld_other, head_dim, seq_len, row_dot, stream=None):
    _check(lib().pw_op_gemm_rowdot(M, N, K, _p(A), lda, _p(B), ldb, _p(C), ldc, _p(other), ld_other, head_dim, seq_len,
                                   _p(row_dot), _stream(stream)))


def op_attention_fwd(qkv, B, S, H, dh, o, lse, stream=None):
    _check(lib().pw_op_attention_fwd(_p(qkv), B, S, H, dh, _p(o), _p(lse), _stream(stream)))


def op_attention_bwd(qkv, o, dout, lse, B, S, H, dh, dqkv, delta, stream=None):
    _check(lib().pw_op_attention_bwd(_p(qkv), _p(o), _p(dout), _p(lse), B, S, H, dh, _p(dqkv), _p(delta),
                                     _stream(stream)))


def op_status():
    c, s = ctypes.c_int(), ctypes.c_int()
    _check(lib().pw_op_status(ctypes.byref(c), ctypes.byref(s)))
    return c.value, s.value


TUNE_PDL, TUNE_GEMM_PAIR, TUNE_GEMM_BN, TUNE_GEMM_SPLIT, TUNE_GEMM_SPLIT_MIN_K, TUNE_FAIL_LAUNCH, TUNE_NVTX = range(7)
LOG_OFF, LOG_ERROR, LOG_INFO = range(3)
LOG_FN = ctypes.CFUNCTYPE(None, ctypes.c_int, ctypes.c_char_p, ctypes.c_void_p)


def set_tuning(knob: int, value: int):
    """Process-wide tuning knob (see pw_set_tuning in include/pw.h)."""
    _check(lib().pw_set_tuning(int(knob), int(value)))


_log_keepalive = None


def set_log(level: int, fn=None):
    """pw_set_log: fn(level, message) or None for stderr; the ctypes thunk is kept alive here."""
    global _log_keepalive
    thunk = LOG_FN(lambda lv, msg, user: fn(lv, msg.decode())) if fn is not None else LOG_FN(0)
    lib().pw_set_log.argtypes = [ctypes.c_int, LOG_FN, ctypes.c_void_p]
    _check(lib().pw_set_log(int(level), thunk, None))
    _log_keepalive = thunk


def get_tuning(knob: int) -> int:
    v = ctypes.c_int(0)
    _check(lib().pw_get_tuning(int(knob), ctypes.byref(v)))
    return v.value


def op_status_reset():
    _check(lib().pw_op_status_reset())


def op_selftest_wait_timeout(limit_cycles=2_000_000, stream=None) -> int:
    """Runs the bounded-wait self-test; returns 1 if the kernel's wait gave up and the kernel returned."""
    r = ctypes.c_int(0)
    _check(lib().pw_op_selftest_wait_timeout(limit_cycles, ctypes.byref(r), _stream(stream)))
    return r.value


def op_affine_f32(x, scale, shift, y, stream=None):
    _check(lib().pw_op_affine_f32(_p(x), x.numel(), scale, shift, _p(y), _stream(stream)))


def sgd_apply(items, lr, grad_scale=1.0, init_master=False, stream=None):
    """items: (param bf16, master fp32, grad fp32) device tensors of equal element counts.
    master -= lr * grad_scale * grad and param = bf16(master), in place, for every item."""
    arr = (ApplyItem * max(len(items), 1))()
    for i, (p, m, g) in enumerate(items):
        assert p.numel() == m.numel() == g.numel(), "param, master and grad must have the same number of elements"
        assert p.is_contiguous() and m.is_contiguous() and g.is_contiguous()
        assert p.element_size() == 2 and m.element_size() == 4 and g.element_size() == 4
        arr[i] = ApplyItem(_p(p), _p(m), _p(g), p.numel())
    _check(lib().pw_sgd_apply(arr, len(items), lr, grad_scale, int(bool(init_master)), _stream(stream)))


def dp_slice(n_total, world, rank):
    """Elements [lo, hi) of the flat index space that replica `rank` owns (host arithmetic only)."""
    lo, hi = ctypes.c_int64(), ctypes.c_int64()
    _check(lib().pw_dp_slice(n_total, world, rank, ctypes.byref(lo), ctypes.byref(hi)))
    return lo.value, hi.value


def dp_reduce_apply(rank, grad_ptrs, param_ptrs, master_slice, n_total, lr, grad_scale, init_master=False, stream=None):
    """grad_ptrs / param_ptrs: device addresses (ints) of every replica's flat buffers, in rank order."""
    world = len(grad_ptrs)
    assert len(param_ptrs) == world
    g = (ctypes.c_void_p * world)(*grad_ptrs)
    p = (ctypes.c_void_p * world)(*param_ptrs)
    _check(lib().pw_dp_reduce_apply(rank, world, g, p, _p(master_slice), n_total, lr, grad_scale, int(bool(init_master)),
                                    _stream(stream)))


def shared_alloc(nbytes):
    """(device address, 64-byte handle) of a new device buffer that other processes can map."""
    ptr, h = ctypes.c_void_p(), IpcHandle()
    _check(lib().pw_shared_alloc(nbytes, ctypes.byref(ptr), ctypes.byref(h)))
    return ptr.value, bytes(h.bytes)


def shared_free(ptr):
    _check(lib().pw_shared_free(ptr))


def shared_open(handle: bytes):
    h = IpcHandle()
    ctypes.memmove(h.bytes, handle, 64)
    ptr = ctypes.c_void_p()
    _check(lib().pw_shared_open(ctypes.byref(h), ctypes.byref(ptr)))
    return ptr.value


def shared_close(ptr):
    _check(lib().pw_shared_close(ptr))
