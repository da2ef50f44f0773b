"""CPU oracle for the decoder-layer hot path.  TEST INFRASTRUCTURE ONLY.

A thin numpy/ctypes front end over ``pw_oracle.c`` (plain C loops, compiled
once as float and once as double).  Only the tests, the smoke entry and the
CPU-baseline leg of the benchmark may import this package; the CUDA library
and its Python binding never do, and this package never imports them.

The paper (Section 5.3) describes the workload only by its sizes, so the
arithmetic is the textbook definition of a pre-LN, causal, decoder-only
Transformer layer; see the header of ``pw_oracle.c`` for what pins it.

All arrays are C-contiguous numpy arrays of the oracle's working precision
(``np.float32`` for ``Oracle('f32')``, ``np.float64`` for ``Oracle('f64')``).
Inputs that are meant to be bf16 values must be rounded by the caller first.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pw_oracle.c")
_BUILD = os.path.join(_HERE, "_build")

PARAM_NAMES = ("ln1_gamma", "ln1_beta", "w_qkv", "b_qkv", "w_o", "b_o",
               "ln2_gamma", "ln2_beta", "w_fc1", "b_fc1", "w_fc2", "b_fc2")
SAVED_NAMES = ("h1", "qkv", "o", "x1", "h2", "u", "a", "lse", "mu1", "r1", "mu2", "r2")
ACT_GELU_ERF = 0
ACT_GELU_TANH = 1


@dataclass(frozen=True)
class Dims:
    """Static shape of one layer call: B sequences of S tokens, d = H*dh, MLP width F."""
    B: int
    S: int
    d: int
    H: int
    dh: int
    F: int
    eps: float = 1e-5
    act: int = ACT_GELU_ERF

    @property
    def T(self) -> int:
        return self.B * self.S

    def param_shapes(self):
        d, F = self.d, self.F
        return ((d,), (d,), (3 * d, d), (3 * d,), (d, d), (d,), (d,), (d,), (F, d), (F,), (d, F), (d,))

    def saved_shapes(self):
        T, d, F = self.T, self.d, self.F
        return ((T, d), (T, 3 * d), (T, d), (T, d), (T, d), (T, F), (T, F),
                (self.B, self.H, self.S), (T,), (T,), (T,), (T,))


def _cpu_tag() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    return line
    except OSError:
        pass
    return "unknown"


def build(verbose: bool = False) -> dict:
    """Compile pw_oracle.c for float and double; returns {'f32': path, 'f64': path}.

    The shared objects are keyed by a hash of the source and of this host's CPU
    flags, so an object built on another machine is never loaded here.
    """
    with open(_SRC, "rb") as f:
        key = hashlib.sha1(f.read() + _cpu_tag().encode()).hexdigest()[:12]
    os.makedirs(_BUILD, exist_ok=True)
    out = {}
    for suf, real in (("f32", "float"), ("f64", "double")):
        so = os.path.join(_BUILD, f"libpw_oracle_{suf}_{key}.so")
        if not os.path.exists(so):
            tmp = so + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=gnu99",
                   f"-DREAL={real}", f"-DSUF={suf}", _SRC, "-o", tmp, "-lm"]
            if verbose:
                print(" ".join(cmd))
            subprocess.run(cmd, check=True)
            os.replace(tmp, so)
        out[suf] = so
    return out


def host_threads() -> int:
    """Number of OpenMP threads the oracle will use (the cores this process may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


class Oracle:
    def __init__(self, precision: str = "f64"):
        assert precision in ("f32", "f64")
        self.suf = precision
        self.dtype = np.float32 if precision == "f32" else np.float64
        self._lib = ctypes.CDLL(build()[precision])

    # -- helpers --
    def _a(self, x):
        a = np.ascontiguousarray(x, dtype=self.dtype)
        return a

    def _p(self, a):
        return a.ctypes.data_as(ctypes.c_void_p)

    def _fn(self, name):
        return getattr(self._lib, f"{name}_{self.suf}")

    def _ptr_array(self, arrays):
        arr = (ctypes.c_void_p * len(arrays))()
        for i, a in enumerate(arrays):
            arr[i] = a.ctypes.data
        return arr

    # -- steps --
    def ln_fwd(self, x, gamma, beta, eps=1e-5):
        x, gamma, beta = self._a(x), self._a(gamma), self._a(beta)
        T, d = x.shape
        h = np.empty_like(x)
        mu = np.empty(T, self.dtype)
        r = np.empty(T, self.dtype)
        self._fn("pwo_ln_fwd")(self._p(x), self._p(gamma), self._p(beta), ctypes.c_long(T), ctypes.c_long(d),
                               ctypes.c_double(eps), self._p(h), self._p(mu), self._p(r))
        return h, mu, r

    def ln_bwd(self, dh, x, mu, rstd, gamma):
        dh, x, mu, rstd, gamma = map(self._a, (dh, x, mu, rstd, gamma))
        T, d = x.shape
        dx = np.empty_like(x)
        dg = np.empty(d, self.dtype)
        db = np.empty(d, self.dtype)
        self._fn("pwo_ln_bwd")(self._p(dh), self._p(x), self._p(mu), self._p(rstd), self._p(gamma),
                               ctypes.c_long(T), ctypes.c_long(d), self._p(dx), self._p(dg), self._p(db))
        return dx, dg, db

    def linear_fwd(self, x, W, b=None):
        x, W = self._a(x), self._a(W)
        T, K = x.shape
        N = W.shape[0]
        assert W.shape == (N, K)
        bb = self._a(b) if b is not None else None
        out = np.empty((T, N), self.dtype)
        self._fn("pwo_linear_fwd")(self._p(x), self._p(W), self._p(bb) if bb is not None else None,
                                   ctypes.c_long(T), ctypes.c_long(K), ctypes.c_long(N), self._p(out))
        return out

    def linear_bwd(self, x, W, dout):
        x, W, dout = self._a(x), self._a(W), self._a(dout)
        T, K = x.shape
        N = W.shape[0]
        dx = np.empty((T, K), self.dtype)
        dW = np.empty((N, K), self.dtype)
        db = np.empty(N, self.dtype)
        self._fn("pwo_linear_bwd")(self._p(x), self._p(W), self._p(dout), ctypes.c_long(T), ctypes.c_long(K),
                                   ctypes.c_long(N), self._p(dx), self._p(dW), self._p(db))
        return dx, dW, db

    def gelu_fwd(self, u, act=ACT_GELU_ERF):
        u = self._a(u)
        a = np.empty_like(u)
        self._fn("pwo_gelu_fwd")(self._p(u), ctypes.c_long(u.size), ctypes.c_int(act), self._p(a))
        return a

    def gelu_bwd(self, u, da, act=ACT_GELU_ERF):
        u, da = self._a(u), self._a(da)
        du = np.empty_like(u)
        self._fn("pwo_gelu_bwd")(self._p(u), self._p(da), ctypes.c_long(u.size), ctypes.c_int(act), self._p(du))
        return du

    def attn_fwd(self, qkv, B, S, H, dh, want_probs=False):
        qkv = self._a(qkv)
        d = H * dh
        assert qkv.shape == (B * S, 3 * d)
        o = np.empty((B * S, d), self.dtype)
        lse = np.empty((B, H, S), self.dtype)
        probs = np.empty((B, H, S, S), self.dtype) if want_probs else None
        self._fn("pwo_attn_fwd")(self._p(qkv), ctypes.c_long(B), ctypes.c_long(S), ctypes.c_long(H),
                                 ctypes.c_long(dh), self._p(o), self._p(lse),
                                 self._p(probs) if want_probs else None)
        return (o, lse, probs) if want_probs else (o, lse)

    def attn_bwd(self, qkv, dout, B, S, H, dh):
        qkv, dout = self._a(qkv), self._a(dout)
        dqkv = np.empty_like(qkv)
        self._fn("pwo_attn_bwd")(self._p(qkv), self._p(dout), ctypes.c_long(B), ctypes.c_long(S),
                                 ctypes.c_long(H), ctypes.c_long(dh), self._p(dqkv))
        return dqkv

    # -- the layer --
    def _dims_args(self, D: Dims):
        return [ctypes.c_long(v) for v in (D.B, D.S, D.d, D.H, D.dh, D.F)]

    def layer_fwd(self, D: Dims, params, x):
        """params: sequence of 12 arrays in PARAM_NAMES order.  Returns (y, saved dict)."""
        assert D.H * D.dh == D.d
        ps = [self._a(p) for p in params]
        for p, shp in zip(ps, D.param_shapes()):
            assert p.shape == shp, (p.shape, shp)
        x = self._a(x).reshape(D.T, D.d)
        saved = [np.empty(shp, self.dtype) for shp in D.saved_shapes()]
        y = np.empty((D.T, D.d), self.dtype)
        self._fn("pwo_layer_fwd")(*self._dims_args(D), ctypes.c_double(D.eps), ctypes.c_int(D.act),
                                  self._ptr_array(ps), self._p(x), self._ptr_array(saved), self._p(y))
        return y, dict(zip(SAVED_NAMES, saved))

    def layer_bwd(self, D: Dims, params, x, saved, dy, grads=None, accumulate=False):
        """Returns (dx, grads list in PARAM_NAMES order).  With accumulate, adds into ``grads``."""
        ps = [self._a(p) for p in params]
        x = self._a(x).reshape(D.T, D.d)
        dy = self._a(dy).reshape(D.T, D.d)
        sv = [self._a(saved[n]) for n in SAVED_NAMES]
        if grads is None:
            assert not accumulate
            grads = [np.zeros(shp, self.dtype) for shp in D.param_shapes()]
        else:
            for g, shp in zip(grads, D.param_shapes()):
                assert g.shape == shp and g.dtype == self.dtype and g.flags.c_contiguous
        dx = np.empty((D.T, D.d), self.dtype)
        self._fn("pwo_layer_bwd")(*self._dims_args(D), ctypes.c_int(D.act), self._ptr_array(ps), self._p(x),
                                  self._ptr_array(sv), self._p(dy), self._p(dx), self._ptr_array(grads),
                                  ctypes.c_int(1 if accumulate else 0))
        return dx, grads

    # -- a pipeline stage: L layers, M micro-batches, gradients summed over micro-batches --
    def chain(self, D: Dims, params_per_layer, xs, dys, handoff=None):
        """Forward through all layers then backward in reverse, for each micro-batch.

        ``handoff`` (optional) is applied to every tensor passed between layers
        (y of layer l -> x of layer l+1, dx of layer l+1 -> dy of layer l); the
        tests pass a bf16 round-trip there to mirror a bf16 hand-off.  Returns
        (ys, dxs, grads[L][12]).
        """
        L = len(params_per_layer)
        grads = [[np.zeros(shp, self.dtype) for shp in D.param_shapes()] for _ in range(L)]
        ys, dxs = [], []
        for m, (x, dy) in enumerate(zip(xs, dys)):
            acts, saves = [self._a(x).reshape(D.T, D.d)], []
            for l in range(L):
                y, sv = self.layer_fwd(D, params_per_layer[l], acts[-1])
                if handoff is not None:
                    y = self._a(handoff(y))
                acts.append(y)
                saves.append(sv)
            g = self._a(dy).reshape(D.T, D.d)
            for l in reversed(range(L)):
                g, _ = self.layer_bwd(D, params_per_layer[l], acts[l], saves[l], g, grads[l], accumulate=(m > 0))
                if handoff is not None:
                    g = self._a(handoff(g))
            ys.append(acts[-1])
            dxs.append(g)
        return ys, dxs, grads

    # -- first and last layer of the language model (embedding lookup, tied softmax head) --
    def embed_fwd(self, ids, E):
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        E = self._a(E)
        T, d = ids.size, E.shape[1]
        assert ids.min() >= 0 and ids.max() < E.shape[0]
        x0 = np.empty((T, d), self.dtype)
        self._fn("pwo_embed_fwd")(self._p(ids), self._p(E), ctypes.c_long(T), ctypes.c_long(d), self._p(x0))
        return x0

    def embed_bwd(self, ids, dx0, dE):
        """dE[ids[t]] += dx0[t] (in place; dE is an array of the oracle's precision)."""
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        dx0 = self._a(dx0)
        assert dE.dtype == self.dtype and dE.flags.c_contiguous
        T, d = dx0.shape
        self._fn("pwo_embed_bwd")(self._p(ids), self._p(dx0), ctypes.c_long(T), ctypes.c_long(d), self._p(dE))
        return dE

    def head_fwd(self, hf, E, labels, want_logits=False):
        """Returns (loss, lse[T]) or (loss, lse, logits[T,V])."""
        hf, E = self._a(hf), self._a(E)
        labels = np.ascontiguousarray(labels, dtype=np.int32)
        T, d = hf.shape
        V = E.shape[0]
        assert E.shape == (V, d) and labels.size == T and labels.min() >= 0 and labels.max() < V
        lse = np.empty(T, self.dtype)
        loss = np.zeros(1, self.dtype)
        logits = np.empty((T, V), self.dtype) if want_logits else None
        self._fn("pwo_head_fwd")(self._p(hf), self._p(E), self._p(labels), ctypes.c_long(T), ctypes.c_long(d),
                                 ctypes.c_long(V), self._p(logits) if want_logits else None, self._p(lse), self._p(loss))
        return (float(loss[0]), lse, logits) if want_logits else (float(loss[0]), lse)

    def head_bwd(self, hf, E, labels, lse, dE, want_dlogits=False):
        """Returns dhf (and dlogits); adds the head's part of the tied gradient into dE."""
        hf, E, lse = self._a(hf), self._a(E), self._a(lse)
        labels = np.ascontiguousarray(labels, dtype=np.int32)
        T, d = hf.shape
        V = E.shape[0]
        assert dE.shape == (V, d) and dE.dtype == self.dtype and dE.flags.c_contiguous
        dhf = np.empty((T, d), self.dtype)
        dz = np.empty((T, V), self.dtype) if want_dlogits else None
        self._fn("pwo_head_bwd")(self._p(hf), self._p(E), self._p(labels), self._p(lse), ctypes.c_long(T),
                                 ctypes.c_long(d), ctypes.c_long(V), self._p(dhf), self._p(dE),
                                 self._p(dz) if want_dlogits else None)
        return (dhf, dz) if want_dlogits else dhf

    def lm_step(self, D: Dims, params_per_layer, E, lnf_gamma, lnf_beta, ids, labels, handoff=None):
        """One training step of the small decoder LM: embedding -> L layers -> final LayerNorm ->
        tied softmax head -> mean cross-entropy, and its backward.

        Returns a dict: loss, grads (per layer, PARAM_NAMES order), dE (embedding + head parts),
        dlnf_gamma, dlnf_beta, and the intermediates x0, hL (last layer output), hf, lse.
        ``handoff`` as in chain().
        """
        L = len(params_per_layer)
        E = self._a(E)
        acts, saves = [self.embed_fwd(ids, E)], []
        for l in range(L):
            y, sv = self.layer_fwd(D, params_per_layer[l], acts[-1])
            if handoff is not None:
                y = self._a(handoff(y))
            acts.append(y)
            saves.append(sv)
        hf, mu, r = self.ln_fwd(acts[-1], lnf_gamma, lnf_beta, D.eps)
        if handoff is not None:
            hf = self._a(handoff(hf))
        loss, lse = self.head_fwd(hf, E, labels)
        dE = np.zeros_like(E)
        dhf = self.head_bwd(hf, E, labels, lse, dE)
        if handoff is not None:
            dhf = self._a(handoff(dhf))
        g, dg, db = self.ln_bwd(dhf, acts[-1], mu, r, lnf_gamma)
        if handoff is not None:
            g = self._a(handoff(g))
        grads = [None] * L
        for l in reversed(range(L)):
            g, grads[l] = self.layer_bwd(D, params_per_layer[l], acts[l], saves[l], g)
            if handoff is not None:
                g = self._a(handoff(g))
        self.embed_bwd(ids, g, dE)
        return {"loss": loss, "grads": grads, "dE": dE, "dlnf_gamma": dg, "dlnf_beta": db,
                "x0": acts[0], "hL": acts[-1], "hf": hf, "lse": lse, "dx0": g}

    # -- the element-wise computations of the Figure 2 program --
    def affine(self, x, scale, shift):
        x = self._a(x)
        y = np.empty_like(x)
        self._fn("pwo_affine")(self._p(x), ctypes.c_long(x.size), ctypes.c_double(scale), ctypes.c_double(shift), self._p(y))
        return y

    # -- gradient apply (plain SGD on a master copy; bf16 working copy) --
    def round_bf16(self, x):
        """x rounded to bf16 (round to nearest, ties to even), kept in the working precision."""
        x = self._a(x)
        return self.sgd_apply(x, np.zeros_like(x), 0.0)[1]            # a step of rate zero only rounds

    def sgd_apply(self, master, grad, lr, grad_scale=1.0):
        """(master - lr * grad_scale * grad, that rounded to bf16); the inputs are not modified."""
        m = self._a(master).copy()
        g = self._a(grad)
        assert m.shape == g.shape
        p = np.empty_like(m)
        self._fn("pwo_sgd_apply")(self._p(m), self._p(g), ctypes.c_long(m.size), ctypes.c_double(lr),
                                  ctypes.c_double(grad_scale), self._p(p))
        return m, p

    def dp_sgd_apply(self, master, grads_per_rank, lr, grad_scale=1.0):
        """Data-parallel form of the gradient apply: every replica's gradient of the same tensor is
        added up (in rank order) and the sum is applied once; all replicas then hold the same
        parameters.  Returns (new master, bf16 working copy)."""
        total = self._a(grads_per_rank[0]).copy()
        for g in grads_per_rank[1:]:
            total = total + self._a(g)
        return self.sgd_apply(master, total, lr, grad_scale)

    def figure2_program(self, v):
        """f(v) = (b(a(v)), a(c(a(v)))) with a(x) = 2x, b(x) = x + 1, c(x) = x / 2 (Figure 2)."""
        a = lambda t: self.affine(t, 2.0, 0.0)
        b = lambda t: self.affine(t, 1.0, 1.0)
        c = lambda t: self.affine(t, 0.5, 0.0)
        return b(a(v)), a(c(a(v)))

