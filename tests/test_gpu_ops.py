"""GPU parity of the single steps (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

from tests.gpu_util import (ACT_TOL, ELEM_ACT, ELEM_F32, ELEM_GRAD, GRAD_TOL, bf16_randn, elem_check, guard_alloc, np64,
                            rel_l2)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()          # raises loudly if the library is not built
    return binding


def _status_ok(pw):
    code, site = pw.op_status()
    assert code == 0, f"device status {code} at site {site}"


# ------------------------------------------------------------------------------------------ GEMM
def test_gemm_tn_integer_exact(pw):
    """Small integers are exact in bf16 and in the fp32 accumulator: any mis-tiled block shows up exactly."""
    g = torch.Generator().manual_seed(1)
    M, N, K = 384, 520, 64
    A = torch.randint(-2, 3, (M, K), generator=g).to(torch.bfloat16)
    B = torch.randint(-2, 3, (N, K), generator=g).to(torch.bfloat16)
    C, check = guard_alloc((M, N), torch.bfloat16)
    pw.op_gemm(pw.GEMM_TN, pw.EPI_NONE, M, N, K, A.cuda(), K, B.cuda(), K, C, N)
    torch.cuda.synchronize()
    _status_ok(pw)
    check()
    want = A.double() @ B.double().T
    assert torch.equal(C.double().cpu(), want)


SHAPES = [(392, 520, 200), (128, 256, 64), (1000, 768, 1032)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("epi", ["none", "bias", "bias_resid", "bias_gelu"])
def test_gemm_tn_epilogues(pw, oracle64, M, N, K, epi):
    g = torch.Generator().manual_seed(2)
    A, W = bf16_randn((M, K), g), bf16_randn((N, K), g, 0.1)
    bias, R = bf16_randn((N,), g), bf16_randn((M, N), g)
    C, check = guard_alloc((M, N), torch.bfloat16)
    aux, check2 = guard_alloc((M, N), torch.bfloat16)
    code = {"none": pw.EPI_NONE, "bias": pw.EPI_BIAS, "bias_resid": pw.EPI_BIAS_RESID, "bias_gelu": pw.EPI_BIAS_GELU}[epi]
    pw.op_gemm(pw.GEMM_TN, code, M, N, K, A.cuda(), K, W.cuda(), K, C, N, bias=bias.cuda(),
               aux_in=R.cuda() if epi == "bias_resid" else None, ld_aux=N,
               aux_out=aux if epi == "bias_gelu" else None)
    torch.cuda.synchronize()
    _status_ok(pw)
    check(); check2()
    want = oracle64.linear_fwd(np64(A), np64(W), np64(bias) if epi != "none" else None)
    if epi == "bias_resid":
        want = want + np64(R)
    assert rel_l2(C, want) < ACT_TOL
    if epi == "bias_gelu":
        assert rel_l2(aux, oracle64.gelu_fwd(want)) < ACT_TOL


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("epi", ["none", "dgelu"])
def test_gemm_nn_dgrad(pw, oracle64, M, N, K, epi):
    """C[M,N] = A[M,K] B[K,N]  (dx = dy W with W stored [out=K, in=N])."""
    g = torch.Generator().manual_seed(3)
    A, W = bf16_randn((M, K), g), bf16_randn((K, N), g, 0.1)
    U = bf16_randn((M, N), g)
    C, check = guard_alloc((M, N), torch.bfloat16)
    pw.op_gemm(pw.GEMM_NN, pw.EPI_DGELU if epi == "dgelu" else pw.EPI_NONE, M, N, K, A.cuda(), K, W.cuda(), N, C, N,
               aux_in=U.cuda() if epi == "dgelu" else None, ld_aux=N)
    torch.cuda.synchronize()
    _status_ok(pw)
    check()
    dx, _, _ = oracle64.linear_bwd(np.zeros((M, N)), np64(W), np64(A))   # dx[t][n] = sum_k dout[t][k] W[k][n]
    if epi == "dgelu":
        dx = oracle64.gelu_bwd(np64(U), dx)
    assert rel_l2(C, dx) < GRAD_TOL


@pytest.mark.parametrize("B,S,H,dh,K", [(2, 128, 4, 128, 512), (3, 128, 6, 64, 384), (1, 640, 3, 128, 384), (1, 128, 2, 64, 128),
                                        (4, 256, 16, 128, 2048)])
def test_gemm_rowdot_epilogue(pw, oracle64, B, S, H, dh, K):
    """dout = dx1 Wo with delta[b][h][s] = sum over head h's columns of dout * o taken in the epilogue;
    the same delta then drives pw_op_attention_bwd (o = None) to the same dqkv as the three-kernel call."""
    g = torch.Generator().manual_seed(31)
    M, N = B * S, H * dh
    A, W = bf16_randn((M, K), g), bf16_randn((K, N), g, 0.1)
    O = bf16_randn((M, N), g)
    C, check = guard_alloc((M, N), torch.bfloat16)
    delta, check_d = guard_alloc((B, H, S), torch.float32)
    pw.op_gemm_rowdot(M, N, K, A.cuda(), K, W.cuda(), N, C, N, O.cuda(), N, dh, S, delta)
    torch.cuda.synchronize()
    _status_ok(pw)
    check(); check_d()
    dout, _, _ = oracle64.linear_bwd(np.zeros((M, N)), np64(W), np64(A))     # dout[t][n] = sum_k A[t][k] W[k][n]
    assert rel_l2(C, dout) < GRAD_TOL
    elem_check(C, dout, "dout", **ELEM_GRAD)
    want = (dout * np64(O)).reshape(B, S, H, dh).sum(-1).transpose(0, 2, 1)  # [B, H, S]
    assert rel_l2(delta, want) < 1e-4
    elem_check(delta, want, "delta", **ELEM_F32)
    # bitwise repeatable
    C2, d2 = torch.empty_like(C), torch.empty_like(delta)
    pw.op_gemm_rowdot(M, N, K, A.cuda(), K, W.cuda(), N, C2, N, O.cuda(), N, dh, S, d2)
    torch.cuda.synchronize()
    assert torch.equal(C, C2) and torch.equal(delta, d2)
    if S % 128 == 0:
        qkv = bf16_randn((M, 3 * N), g).cuda()
        o_dev, lse = torch.empty((M, N), dtype=torch.bfloat16, device="cuda"), torch.empty((B, H, S), device="cuda")
        pw.op_attention_fwd(qkv, B, S, H, dh, o_dev, lse)
        dq_a, dq_b = torch.empty_like(qkv), torch.empty_like(qkv)
        dl = torch.empty((B, H, S), device="cuda")
        pw.op_gemm_rowdot(M, N, K, A.cuda(), K, W.cuda(), N, C2, N, o_dev, N, dh, S, d2)
        pw.op_attention_bwd(qkv, o_dev, C2, lse, B, S, H, dh, dq_a, dl)        # delta by the row-dot kernel (from bf16 dout)
        pw.op_attention_bwd(qkv, None, C2, lse, B, S, H, dh, dq_b, d2)         # delta from the GEMM epilogue (from fp32 dout)
        torch.cuda.synchronize()
        _status_ok(pw)
        assert rel_l2(d2, dl) < 5e-3
        assert rel_l2(dq_b, dq_a) < 5e-3


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("accumulate", [False, True])
def test_gemm_nt_wgrad(pw, oracle64, M, N, K, accumulate):
    """C[M,N] (+)= A[K,M]^T B[K,N]  (dW = dy^T x), fp32 output."""
    g = torch.Generator().manual_seed(4)
    A, B = bf16_randn((K, M), g), bf16_randn((K, N), g)
    C, check = guard_alloc((M, N), torch.float32)
    C0 = torch.randn((M, N), generator=g)
    C.copy_(C0)
    pw.op_gemm(pw.GEMM_NT, pw.EPI_F32, M, N, K, A.cuda(), M, B.cuda(), N, C, N, accumulate=accumulate)
    torch.cuda.synchronize()
    _status_ok(pw)
    check()
    _, dW, _ = oracle64.linear_bwd(np64(B), np.zeros((M, N)), np64(A))   # dW[m][n] = sum_k A[k][m] B[k][n]
    if accumulate:
        dW = dW + np64(C0)
    assert rel_l2(C, dW) < 1e-5


def test_gemm_is_deterministic(pw):
    g = torch.Generator().manual_seed(5)
    M, N, K = 640, 512, 448
    A, W = bf16_randn((M, K), g).cuda(), bf16_randn((N, K), g).cuda()
    C1 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    C2 = torch.empty_like(C1)
    pw.op_gemm(pw.GEMM_TN, pw.EPI_NONE, M, N, K, A, K, W, K, C1, N)
    pw.op_gemm(pw.GEMM_TN, pw.EPI_NONE, M, N, K, A, K, W, K, C2, N)
    torch.cuda.synchronize()
    assert torch.equal(C1, C2)


def test_gemm_rejects_bad_arguments(pw):
    A = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pw.PwError):
        pw.op_gemm(pw.GEMM_TN, pw.EPI_NONE, 128, 128, 60, A, 64, A, 64, A, 128)        # K not a multiple of 8
    with pytest.raises(pw.PwError):
        pw.op_gemm(pw.GEMM_TN, pw.EPI_BIAS, 128, 128, 64, A, 64, A, 64, A, 128)        # bias missing
    with pytest.raises(pw.PwError):
        pw.op_gemm(pw.GEMM_NT, pw.EPI_BIAS, 128, 128, 64, A, 64, A, 64, A, 128, bias=A)  # unsupported combination


# ------------------------------------------------------------------------------------------ LayerNorm / column sums
@pytest.mark.parametrize("T,d", [(77, 256), (130, 1024), (515, 2048), (70, 4096), (33, 8192), (64, 1536)])
def test_layernorm_fwd_bwd(pw, oracle64, T, d):
    g = torch.Generator().manual_seed(6)
    x = bf16_randn((T, d), g, 2.0) + 0.5
    x = x.to(torch.bfloat16)
    gamma = (1 + 0.2 * torch.randn(d, generator=g)).to(torch.bfloat16)
    beta = (0.2 * torch.randn(d, generator=g)).to(torch.bfloat16)
    dh, resid = bf16_randn((T, d), g), bf16_randn((T, d), g)
    h, check_h = guard_alloc((T, d), torch.bfloat16)
    mu = torch.empty(T, device="cuda"); r = torch.empty(T, device="cuda")
    pw.op_layernorm_fwd(x.cuda(), gamma.cuda(), beta.cuda(), 1e-5, h, mu, r)
    torch.cuda.synchronize()
    check_h()
    hw, muw, rw = oracle64.ln_fwd(np64(x), np64(gamma), np64(beta), 1e-5)
    assert rel_l2(h, hw) < ACT_TOL and rel_l2(mu, muw) < 1e-5 and rel_l2(r, rw) < 1e-5
    elem_check(h, hw, "h", **ELEM_ACT)
    elem_check(mu, muw, "mu", **ELEM_F32)
    elem_check(r, rw, "rstd", **ELEM_F32)

    dx, check_dx = guard_alloc((T, d), torch.bfloat16)
    outs = [torch.full((d,), 3.0, device="cuda") for _ in range(4)]
    part = torch.empty(pw.op_layernorm_bwd_scratch_bytes(T, d), dtype=torch.uint8, device="cuda")
    for acc in (False, True):
        pw.op_layernorm_bwd(dh.cuda(), x.cuda(), mu, r, gamma.cuda(), resid.cuda(), dx, outs[0], outs[1], outs[2],
                            outs[3], acc, part)
    torch.cuda.synchronize()
    check_dx()
    dxw, dgw, dbw = oracle64.ln_bwd(np64(dh), np64(x), muw, rw, np64(gamma))
    dxw = dxw + np64(resid)
    assert rel_l2(dx, dxw) < GRAD_TOL
    elem_check(dx, dxw, "dx", **ELEM_GRAD)
    assert rel_l2(outs[0], 2 * dgw) < GRAD_TOL and rel_l2(outs[1], 2 * dbw) < GRAD_TOL   # overwrite, then accumulate
    elem_check(outs[0], 2 * dgw, "dgamma", **ELEM_GRAD)
    elem_check(outs[1], 2 * dbw, "dbeta", **ELEM_GRAD)
    assert rel_l2(outs[2], 2 * np64(resid).sum(0)) < 1e-4
    assert rel_l2(outs[3], 2 * dxw.sum(0)) < GRAD_TOL


@pytest.mark.parametrize("T,N", [(100, 256), (1000, 3072), (777, 8192), (5, 1032)])
def test_colsum(pw, T, N):
    g = torch.Generator().manual_seed(7)
    a = bf16_randn((T, N), g)
    out = torch.full((N,), 1.0, device="cuda")
    part = torch.empty(max(16, pw.op_colsum_scratch_bytes(T, N)), dtype=torch.uint8, device="cuda")
    pw.op_colsum(a.cuda(), out, False, part)
    pw.op_colsum(a.cuda(), out, True, part)
    torch.cuda.synchronize()
    assert rel_l2(out, 2 * np64(a).sum(0)) < 1e-5


# ------------------------------------------------------------------------------------------ attention
@pytest.mark.parametrize("B,S,H,dh", [(2, 128, 2, 64), (2, 384, 3, 64), (1, 256, 2, 128), (2, 640, 1, 128)])
def test_attention_fwd_bwd(pw, oracle64, B, S, H, dh):
    g = torch.Generator().manual_seed(8)
    d = H * dh
    qkv = bf16_randn((B * S, 3 * d), g)
    dout = bf16_randn((B * S, d), g)
    o, check_o = guard_alloc((B * S, d), torch.bfloat16)
    lse, check_l = guard_alloc((B, H, S), torch.float32)
    pw.op_attention_fwd(qkv.cuda(), B, S, H, dh, o, lse)
    torch.cuda.synchronize()
    check_o(); check_l()
    ow, lw = oracle64.attn_fwd(np64(qkv), B, S, H, dh)
    assert rel_l2(o, ow) < ACT_TOL
    elem_check(o, ow, "o", **ELEM_ACT)
    assert np.abs(lse.double().cpu().numpy() - lw).max() < 1e-3

    dqkv, check_d = guard_alloc((B * S, 3 * d), torch.bfloat16)
    delta = torch.empty((B, H, S), device="cuda")
    pw.op_attention_bwd(qkv.cuda(), o, dout.cuda(), lse, B, S, H, dh, dqkv, delta)
    torch.cuda.synchronize()
    _status_ok(pw)
    check_d()
    dw = oracle64.attn_bwd(np64(qkv), np64(dout), B, S, H, dh)
    for name, sl in (("dq", slice(0, d)), ("dk", slice(d, 2 * d)), ("dv", slice(2 * d, 3 * d))):
        assert rel_l2(dqkv[:, sl], dw[:, sl]) < GRAD_TOL, name
        elem_check(dqkv[:, sl], dw[:, sl], name, **ELEM_GRAD)


@pytest.mark.parametrize("S,dh", [(2048, 128), (2048, 64), (4096, 128), (4096, 64)])
def test_attention_long_sequences_every_row(pw, oracle64, S, dh):
    """Sequences of 16 and 32 key tiles (the 2048 tokens of workloads 3 and 4, and twice that): every
    row of o, lse, dq, dk and dv against the oracle, by norm and element by element - the online
    softmax rescales many times, the shared-memory rings wrap, and the work items of different weight
    are drawn heaviest first.  A second backward call must give the same bits."""
    g = torch.Generator().manual_seed(15 + S + dh)
    B, H = 1, 2
    d = H * dh
    qkv = bf16_randn((B * S, 3 * d), g)
    dout = bf16_randn((B * S, d), g)
    o, check_o = guard_alloc((B * S, d), torch.bfloat16)
    lse, check_l = guard_alloc((B, H, S), torch.float32)
    pw.op_attention_fwd(qkv.cuda(), B, S, H, dh, o, lse)
    torch.cuda.synchronize()
    _status_ok(pw)
    check_o(); check_l()
    ow, lw = oracle64.attn_fwd(np64(qkv), B, S, H, dh)
    assert rel_l2(o, ow) < ACT_TOL
    elem_check(o, ow, "o", **ELEM_ACT)
    assert np.abs(lse.double().cpu().numpy() - lw).max() < 1e-3
    dqkv, check_d = guard_alloc((B * S, 3 * d), torch.bfloat16)
    dqkv2 = torch.empty((B * S, 3 * d), dtype=torch.bfloat16, device="cuda")
    delta = torch.empty((B, H, S), device="cuda")
    pw.op_attention_bwd(qkv.cuda(), o, dout.cuda(), lse, B, S, H, dh, dqkv, delta)
    delta.fill_(float("nan"))                          # nothing of the first call may be needed by the second
    pw.op_attention_bwd(qkv.cuda(), o, dout.cuda(), lse, B, S, H, dh, dqkv2, delta)
    torch.cuda.synchronize()
    _status_ok(pw)
    check_d()
    assert torch.equal(dqkv, dqkv2)
    dw = oracle64.attn_bwd(np64(qkv), np64(dout), B, S, H, dh)
    for name, sl in (("dq", slice(0, d)), ("dk", slice(d, 2 * d)), ("dv", slice(2 * d, 3 * d))):
        assert rel_l2(dqkv[:, sl], dw[:, sl]) < GRAD_TOL, name
        elem_check(dqkv[:, sl], dw[:, sl], name, **ELEM_GRAD)


def test_attention_is_causal_and_deterministic(pw):
    g = torch.Generator().manual_seed(9)
    B, S, H, dh = 1, 256, 2, 64
    d = H * dh
    qkv = bf16_randn((B * S, 3 * d), g).cuda()
    o1 = torch.empty((B * S, d), dtype=torch.bfloat16, device="cuda"); o2 = torch.empty_like(o1); o3 = torch.empty_like(o1)
    lse = torch.empty((B, H, S), device="cuda")
    pw.op_attention_fwd(qkv, B, S, H, dh, o1, lse)
    pw.op_attention_fwd(qkv, B, S, H, dh, o2, lse)
    q2 = qkv.clone()
    q2[150:] += 1.0                                    # tokens >= 150 change; outputs at positions < 150 must not
    pw.op_attention_fwd(q2, B, S, H, dh, o3, lse)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2)
    assert torch.equal(o1[:150], o3[:150]) and not torch.equal(o1[150:], o3[150:])


def test_figure2_program_on_a_stream_and_as_a_captured_graph(pw):
    """The paper's Figure 2 worked example, f(v) = (b(a(v)), a(c(a(v)))), a = x*2, b = x+1, c = x/2,
    run through the C ABI: enqueued on a stream and as a captured CUDA graph; both must give the
    values the paper prints."""
    import os
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "figure2_program.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *nums = line.split()
                vals[k] = torch.tensor([float(t) for t in nums], dtype=torch.float32)
    v = vals["v"].cuda()
    t1, t2, out0, out1 = (torch.empty_like(v) for _ in range(4))
    stream = torch.cuda.Stream()

    def program():
        pw.op_affine_f32(v, 2.0, 0.0, t1, stream=stream)        # a(v)
        pw.op_affine_f32(t1, 1.0, 1.0, out0, stream=stream)     # b(a(v))
        pw.op_affine_f32(t1, 0.5, 0.0, t2, stream=stream)       # c(a(v))
        pw.op_affine_f32(t2, 2.0, 0.0, out1, stream=stream)     # a(c(a(v)))

    with torch.cuda.stream(stream):
        program()
    torch.cuda.synchronize()
    assert torch.equal(out0.cpu(), vals["out0"]) and torch.equal(out1.cpu(), vals["out1"])
    out0.zero_(); out1.zero_()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        program()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out0.cpu(), vals["out0"]) and torch.equal(out1.cpu(), vals["out1"])


def test_gemm_random_shapes_all_layouts(pw, oracle64):
    """Twelve seeded random shapes (multiples of 8 between 8 and ~1600, so tile tails in every
    dimension, one-CTA and CTA-pair kernels, partly filled rounds) through every layout."""
    rng = np.random.default_rng(11)
    g = torch.Generator().manual_seed(12)
    for case in range(12):
        M, N, K = (int(8 * rng.integers(1, 200)) for _ in range(3))
        layout = (pw.GEMM_TN, pw.GEMM_NN, pw.GEMM_NT)[case % 3]
        A, Bm = bf16_randn((M, K), g), bf16_randn((K, N), g, 0.1)          # mathematical operands: C = A @ Bm
        want = np64(A) @ np64(Bm)
        if layout == pw.GEMM_TN:
            a_dev, lda, b_dev, ldb = A.cuda(), K, Bm.t().contiguous().cuda(), K      # B stored [N, K]
        elif layout == pw.GEMM_NN:
            a_dev, lda, b_dev, ldb = A.cuda(), K, Bm.cuda(), N                        # B stored [K, N]
        else:
            a_dev, lda, b_dev, ldb = A.t().contiguous().cuda(), M, Bm.cuda(), N      # A stored [K, M]
        f32 = layout == pw.GEMM_NT
        C, check = guard_alloc((M, N), torch.float32 if f32 else torch.bfloat16)
        pw.op_gemm(layout, pw.EPI_F32 if f32 else pw.EPI_NONE, M, N, K, a_dev, lda, b_dev, ldb, C, N)
        torch.cuda.synchronize()
        _status_ok(pw)
        check()
        assert rel_l2(C, want) < (1e-5 if f32 else ACT_TOL), (case, layout, M, N, K)


def test_attention_random_shapes(pw, oracle64):
    """Seeded random (B, S, H, dh): odd and even tile counts, more and fewer work items than SMs."""
    rng = np.random.default_rng(13)
    g = torch.Generator().manual_seed(14)
    for case in range(5):
        B, S, H = int(rng.integers(1, 4)), 128 * int(rng.integers(1, 6)), int(rng.integers(1, 5))
        dh = (64, 128)[case % 2]
        d = H * dh
        qkv = bf16_randn((B * S, 3 * d), g)
        dout = bf16_randn((B * S, d), g)
        o = torch.empty((B * S, d), dtype=torch.bfloat16, device="cuda")
        lse = torch.empty((B, H, S), device="cuda")
        dqkv = torch.empty((B * S, 3 * d), dtype=torch.bfloat16, device="cuda")
        delta = torch.empty((B, H, S), device="cuda")
        pw.op_attention_fwd(qkv.cuda(), B, S, H, dh, o, lse)
        pw.op_attention_bwd(qkv.cuda(), o, dout.cuda(), lse, B, S, H, dh, dqkv, delta)
        torch.cuda.synchronize()
        _status_ok(pw)
        ow, lsew = oracle64.attn_fwd(np64(qkv), B, S, H, dh)
        assert rel_l2(o, ow) < ACT_TOL, (case, B, S, H, dh)
        elem_check(o, ow, f"o case {case}", **ELEM_ACT)
        assert np.allclose(lse.cpu().numpy(), lsew, atol=2e-3), (case, B, S, H, dh)
        dw = oracle64.attn_bwd(np64(qkv), np64(dout), B, S, H, dh)
        assert rel_l2(dqkv, dw) < GRAD_TOL, (case, B, S, H, dh)
        for name, sl in (("dq", slice(0, d)), ("dk", slice(d, 2 * d)), ("dv", slice(2 * d, 3 * d))):
            elem_check(dqkv[:, sl], dw[:, sl], f"{name} case {case}", **ELEM_GRAD)


def test_gemm_tiles_cut_along_k_are_exact_and_reproducible(pw):
    """110 pair tiles on 74 CTA pairs: the 36 tiles of the last round are cut in two along K and the
    halves meet through the scratch (bf16-output GEMMs with K >= 4096 only; the fp32-output layout
    is run for comparison).  Integer operands make every partial sum exact, so the result must be
    the exact product (rounded once to bf16 where the output is bf16), five times in a row (the
    tickets are back at zero after every launch)."""
    g = torch.Generator().manual_seed(9)
    M, N, K = 2560, 2816, 4096
    ri = lambda *s: torch.randint(-2, 3, s, generator=g).to(torch.bfloat16)
    # TN: C = A B^T + bias + residual
    A, B = ri(M, K), ri(N, K)
    bias, resid = ri(N), ri(M, N)
    want = (A.double() @ B.double().T + bias.double() + resid.double()).to(torch.bfloat16)
    Ad, Bd, bd, rd = A.cuda(), B.cuda(), bias.cuda(), resid.cuda()
    for _ in range(5):
        C, check = guard_alloc((M, N), torch.bfloat16)
        pw.op_gemm(pw.GEMM_TN, pw.EPI_BIAS_RESID, M, N, K, Ad, K, Bd, K, C, N, bias=bd, aux_in=rd, ld_aux=N)
        torch.cuda.synchronize()
        _status_ok(pw)
        check()
        assert torch.equal(C.cpu(), want)
    # NN: C = A B  (dgrad: B stored [K, N])
    Bn = ri(K, N)
    want = (A.double() @ Bn.double()).to(torch.bfloat16)
    C, check = guard_alloc((M, N), torch.bfloat16)
    pw.op_gemm(pw.GEMM_NN, pw.EPI_NONE, M, N, K, Ad, K, Bn.cuda(), N, C, N)
    torch.cuda.synchronize()
    _status_ok(pw)
    check()
    assert torch.equal(C.cpu(), want)
    # NT: C (+)= A^T B, fp32 (A stored [K, M], B stored [K, N])
    At = ri(K, M)
    want = At.double().T @ Bn.double()
    C0 = torch.randint(-5, 6, (M, N), generator=g).float()
    for accumulate in (False, True):
        C, check = guard_alloc((M, N), torch.float32)
        C.copy_(C0)
        pw.op_gemm(pw.GEMM_NT, pw.EPI_F32, M, N, K, At.cuda(), M, Bn.cuda(), N, C, N, accumulate=accumulate)
        torch.cuda.synchronize()
        _status_ok(pw)
        check()
        assert torch.equal(C.double().cpu(), want + (C0.double() if accumulate else 0))
    # a GEMM that is not cut still works afterwards
    test_gemm_tn_integer_exact(pw)


@pytest.mark.parametrize("M,N,K", [(2056, 2312, 4104), (4096, 1280, 4096), (1288, 3848, 5000), (2304, 2304, 8200),
                                    (8192, 2048, 4096)])
def test_gemm_cut_tiles_ragged_shapes_are_exact(pw, M, N, K):
    """Shapes whose last round of 256 x 256 tiles keeps at most half of the 74 CTA pairs busy (so its
    tiles are cut along K), with ragged edges in every dimension: integer operands, exact result, for
    the forward layout with the GeLU' -free epilogues and for the data-gradient layout."""
    tiles = -(-M // 256) * -(-N // 256)
    rem = tiles % 74
    assert tiles > 74 and 0 < rem <= 37 and K >= 4096, (tiles, rem)      # the launcher's condition for cutting
    g = torch.Generator().manual_seed(M + N + K)
    ri = lambda *s: torch.randint(-2, 3, s, generator=g).to(torch.bfloat16)
    A, B, Bn, bias = ri(M, K), ri(N, K), ri(K, N), ri(N)
    Ad = A.cuda()
    want = (A.double() @ B.double().T + bias.double()).to(torch.bfloat16)
    C, check = guard_alloc((M, N), torch.bfloat16)
    pw.op_gemm(pw.GEMM_TN, pw.EPI_BIAS, M, N, K, Ad, K, B.cuda(), K, C, N, bias=bias.cuda())
    torch.cuda.synchronize()
    _status_ok(pw)
    check()
    assert torch.equal(C.cpu(), want)
    want = (A.double() @ Bn.double()).to(torch.bfloat16)
    C, check = guard_alloc((M, N), torch.bfloat16)
    pw.op_gemm(pw.GEMM_NN, pw.EPI_NONE, M, N, K, Ad, K, Bn.cuda(), N, C, N)
    torch.cuda.synchronize()
    _status_ok(pw)
    check()
    assert torch.equal(C.cpu(), want)
