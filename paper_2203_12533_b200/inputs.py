"""Seeded synthetic inputs for the decoder-layer hot path.

This module only draws random numbers and rounds them to bf16; it holds none
of the layer's arithmetic, so both the CUDA path and the CPU checker can be
fed from it without sharing any of the method's code.

The five workloads this library is measured on (Section 5.3 of the
paper gives the 3e9-parameter decoder's sizes: model dimension 2048, hidden
dimension 8192, micro-batches of 4 examples, S stages x M micro-batches):

  1  d=256,  4x64 heads,   F=1024,  S=128,  B=2               (tiny parity case)
  2  d=2048, 16x128 heads, F=8192,  S=1024, B=8               (the paper's layer; benchmark workload)
  3  4 layers d=4096, 32x128, F=16384, S=2048, B=4, 16 micro-batches, recompute
  4  d=8192, 64x128 heads, F=32768, S=2048, B=1, weights N(0, 0.01)
  5  12 layers d=1024, 16x64, F=4096, S=1024, B=16 (+ vocabulary 32768 for the LM head)

Recipe.  Everything is drawn on the host with ``torch.Generator`` (CPU), as
fp32 normal deviates, scaled, then rounded to bf16 (round-to-nearest-even).
Layer l of a job with seed s uses generator seed ``s*7919 + 17*l + 1`` and
draws, in this order: w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2, b_fc2
(all N(0, sigma_w)); LayerNorm gammas are 1 and betas 0 unless
``random_ln=True`` (then gamma ~ 1 + N(0, 0.1), beta ~ N(0, 0.1), drawn after
the weights).  Micro-batch m uses seed ``s*7919 + 100003 + m`` and draws
x ~ N(0,1) [B,S,d] then dy ~ N(0,1) [B,S,d].
The language-model workload (5) adds, from seed ``s*7919 + 200003``: the embedding table
E ~ N(0, 0.02) [V,d] (also the output projection: tied), token ids and labels, both independent
uniform integers in [0, V) (int32 [B,S]; the labels are not shifted ids), and the final
LayerNorm's gamma = 1, beta = 0 (``random_ln`` as above).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

PARAM_NAMES = ("ln1_gamma", "ln1_beta", "w_qkv", "b_qkv", "w_o", "b_o",
               "ln2_gamma", "ln2_beta", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


@dataclass(frozen=True)
class Workload:
    name: str
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    seq_len: int
    batch: int
    n_layers: int = 1
    n_microbatches: int = 1
    sigma_w: float = 0.02
    recompute: bool = False
    vocab: int = 0

    @property
    def tokens(self) -> int:
        return self.batch * self.seq_len

    def param_shapes(self):
        d, F = self.d_model, self.d_ff
        return ((d,), (d,), (3 * d, d), (3 * d,), (d, d), (d,), (d,), (d,), (F, d), (F,), (d, F), (d,))

    def model_flops_per_layer_call(self) -> float:
        """fwd+bwd FLOPs of one layer on one micro-batch: 24Td^2 + 12TdF + 7TSd.

        Causal attention is counted at the S(S+1)/2 visible pairs, i.e. the work
        the method has to do, not the masked half."""
        T, d, F, S = self.tokens, self.d_model, self.d_ff, self.seq_len
        gemm = 8.0 * T * d * d + 4.0 * T * d * F
        attn = 4.0 * T * S * d / 2.0 * (1.0 + 1.0 / S)
        return 3.0 * gemm + 3.5 * attn

    def fwd_flops_per_layer_call(self) -> float:
        T, d, F, S = self.tokens, self.d_model, self.d_ff, self.seq_len
        return 8.0 * T * d * d + 4.0 * T * d * F + 4.0 * T * S * d / 2.0 * (1.0 + 1.0 / S)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    1: Workload("cfg1_d256_s128_b2", 256, 4, 64, 1024, 128, 2),
    2: Workload("cfg2_d2048_s1024_b8", 2048, 16, 128, 8192, 1024, 8),
    3: Workload("cfg3_chain4_d4096_s2048_b4_m16", 4096, 32, 128, 16384, 2048, 4, n_layers=4,
                n_microbatches=16, recompute=True),
    4: Workload("cfg4_d8192_s2048_b1", 8192, 64, 128, 32768, 2048, 1, sigma_w=0.01),
    5: Workload("cfg5_lm12_d1024_s1024_b16", 1024, 16, 64, 4096, 1024, 16, n_layers=12, vocab=32768),
}


def _bf16(t: torch.Tensor) -> torch.Tensor:
    return t.to(torch.bfloat16)


def layer_params(w: Workload, seed: int = 0, layer: int = 0, random_ln: bool = False):
    """The 12 parameter tensors of one layer (bf16, CPU), in PARAM_NAMES order."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 7919 + 17 * layer + 1)
    shapes = w.param_shapes()
    out = [None] * 12
    for i in (2, 3, 4, 5, 8, 9, 10, 11):
        out[i] = _bf16(torch.randn(shapes[i], generator=g, dtype=torch.float32) * w.sigma_w)
    for gi, bi in ((0, 1), (6, 7)):
        if random_ln:
            out[gi] = _bf16(1.0 + 0.1 * torch.randn(shapes[gi], generator=g, dtype=torch.float32))
            out[bi] = _bf16(0.1 * torch.randn(shapes[bi], generator=g, dtype=torch.float32))
        else:
            out[gi] = torch.ones(shapes[gi], dtype=torch.bfloat16)
            out[bi] = torch.zeros(shapes[bi], dtype=torch.bfloat16)
    return out


def microbatch(w: Workload, seed: int = 0, m: int = 0):
    """(x, dy) of micro-batch m: bf16 CPU tensors of shape [B, S, d]."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 7919 + 100003 + m)
    shp = (w.batch, w.seq_len, w.d_model)
    x = _bf16(torch.randn(shp, generator=g, dtype=torch.float32))
    dy = _bf16(torch.randn(shp, generator=g, dtype=torch.float32))
    return x, dy


def lm_inputs(w: Workload, seed: int = 0, random_ln: bool = False):
    """(E [V,d] bf16, lnf_gamma [d] bf16, lnf_beta [d] bf16, ids [B,S] int32, labels [B,S] int32), CPU tensors."""
    assert w.vocab > 0
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 7919 + 200003)
    E = _bf16(torch.randn((w.vocab, w.d_model), generator=g, dtype=torch.float32) * 0.02)
    ids = torch.randint(0, w.vocab, (w.batch, w.seq_len), generator=g, dtype=torch.int32)
    labels = torch.randint(0, w.vocab, (w.batch, w.seq_len), generator=g, dtype=torch.int32)
    if random_ln:
        gamma = _bf16(1.0 + 0.1 * torch.randn((w.d_model,), generator=g, dtype=torch.float32))
        beta = _bf16(0.1 * torch.randn((w.d_model,), generator=g, dtype=torch.float32))
    else:
        gamma = torch.ones((w.d_model,), dtype=torch.bfloat16)
        beta = torch.zeros((w.d_model,), dtype=torch.bfloat16)
    return E, gamma, beta, ids, labels

