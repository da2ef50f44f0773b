/*
 * CPU oracle for the decoder-layer hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the checker, not the product: only the tests, the smoke entry
 * and the CPU-baseline leg of the benchmark may build, load or call it.  It
 * shares no code, header, table or constant with the CUDA library and never
 * will; the CUDA library never calls into it.
 *
 * What it computes.  The paper's Section 5.3 workload is a decoder-only
 * Transformer language model described only by its sizes (62 layers, model
 * dimension 2048, hidden dimension 8192, about 3e9 parameters, an embedding
 * layer first and a softmax layer last, micro-batches of 4 examples).  The
 * paper prints no formula for the layer, so each function below is the
 * textbook definition of the operation, written out as plain loops in one
 * working precision (REAL = float or double; the file is compiled once for
 * each) with no blocking, fusion or re-association beyond an explicit SIMD
 * reduction on the innermost dot-product loops.  Readings of everything the
 * paper leaves open (pre-LN placement, biases, erf GeLU, 1/sqrt(dh) scale,
 * causal mask, packing of q/k/v) are listed in the repository's design notes.
 *
 * Pinning.  Every function here is pinned by CPU tests against something
 * other than itself: central finite differences in double, fp64 library
 * routines (layer norm, scaled-dot-product attention, GeLU, autograd),
 * closed forms (one-token attention, equal keys -> prefix means, zeroed
 * output weights -> identity), causality, softmax row sums, LayerNorm moments,
 * linearity of the backward pass, and the parameter-count identity of
 * Section 5.3.  The language-model ends (embedding lookup, tied softmax head with
 * cross-entropy) are pinned by closed forms (zero table -> ln V, gradient rows summing
 * to zero), scipy's logsumexp, torch's cross_entropy + autograd in double, central
 * differences through the whole small-LM step and the initial-loss window of the
 * workload recipe; the Figure 2 program by the values the paper prints; the gradient
 * apply by a library bf16 conversion, the closed form after k equal steps, the exact
 * minimiser of a quadratic and the first-order loss decrease of the small-LM step.
 * Every function in this file has at least one such pin.
 *
 * Layout conventions (all row-major, all REAL):
 *   activations  [T, width], T = B*S tokens, token t = b*S + s
 *   weights      [out_features, in_features]   (y = x W^T + b)
 *   qkv          [T, 3d]: columns [0,d) = q, [d,2d) = k, [2d,3d) = v;
 *                head h occupies columns h*dh .. h*dh+dh-1 of each block
 *   lse          [B, H, S]
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifndef REAL
#error "compile with -DREAL=float -DSUF=f32 or -DREAL=double -DSUF=f64"
#endif
#define CAT_(a, b) a##_##b
#define CAT(a, b) CAT_(a, b)
#define FN(name) CAT(name, SUF)

#define PWO_ACT_GELU_ERF 0
#define PWO_ACT_GELU_TANH 1

/* ---- LayerNorm over the last dimension (biased variance, two passes) ---- */
/* h = gamma * (x - mu) * r + beta,  mu = mean(x),  r = 1/sqrt(var + eps).   */
void FN(pwo_ln_fwd)(const REAL* x, const REAL* gamma, const REAL* beta, long T, long d, double eps,
                    REAL* h, REAL* mu, REAL* rstd)
{
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        const REAL* xr = x + t * d;
        REAL m = 0;
        for (long c = 0; c < d; ++c) m += xr[c];
        m /= (REAL)d;
        REAL v = 0;
        for (long c = 0; c < d; ++c) v += (xr[c] - m) * (xr[c] - m);
        v /= (REAL)d;
        REAL r = (REAL)1 / (REAL)sqrt((double)v + eps);
        for (long c = 0; c < d; ++c) h[t * d + c] = gamma[c] * ((xr[c] - m) * r) + beta[c];
        mu[t] = m;
        rstd[t] = r;
    }
}

/* Backward of LayerNorm.  With xhat = (x - mu) r and g = dh * gamma:
 *   dx = r * ( g - mean(g) - xhat * mean(g * xhat) )
 *   dgamma = sum_t dh * xhat,   dbeta = sum_t dh                              */
void FN(pwo_ln_bwd)(const REAL* dh, const REAL* x, const REAL* mu, const REAL* rstd, const REAL* gamma,
                    long T, long d, REAL* dx, REAL* dgamma, REAL* dbeta)
{
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        REAL m = mu[t], r = rstd[t];
        REAL sg = 0, sgx = 0;
        for (long c = 0; c < d; ++c) {
            REAL xh = (x[t * d + c] - m) * r;
            REAL g = dh[t * d + c] * gamma[c];
            sg += g;
            sgx += g * xh;
        }
        sg /= (REAL)d;
        sgx /= (REAL)d;
        for (long c = 0; c < d; ++c) {
            REAL xh = (x[t * d + c] - m) * r;
            REAL g = dh[t * d + c] * gamma[c];
            dx[t * d + c] = r * (g - sg - xh * sgx);
        }
    }
#pragma omp parallel for schedule(static)
    for (long c = 0; c < d; ++c) {
        REAL a = 0, b = 0;
        for (long t = 0; t < T; ++t) {
            REAL xh = (x[t * d + c] - mu[t]) * rstd[t];
            a += dh[t * d + c] * xh;
            b += dh[t * d + c];
        }
        dgamma[c] = a;
        dbeta[c] = b;
    }
}

/* ---- Linear layer: out[t][n] = b[n] + sum_k x[t][k] W[n][k] ---- */
void FN(pwo_linear_fwd)(const REAL* x, const REAL* W, const REAL* b, long T, long K, long N, REAL* out)
{
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t)
        for (long n = 0; n < N; ++n) {
            const REAL* xr = x + t * K;
            const REAL* wr = W + n * K;
            REAL s = 0;
#pragma omp simd reduction(+ : s)
            for (long k = 0; k < K; ++k) s += xr[k] * wr[k];
            out[t * N + n] = s + (b ? b[n] : (REAL)0);
        }
}

/* Backward of the linear layer:
 *   dx[t][k] = sum_n dout[t][n] W[n][k]
 *   dW[n][k] = sum_t dout[t][n] x[t][k]
 *   db[n]    = sum_t dout[t][n]                                              */
void FN(pwo_linear_bwd)(const REAL* x, const REAL* W, const REAL* dout, long T, long K, long N,
                        REAL* dx, REAL* dW, REAL* db)
{
    if (dx) {
#pragma omp parallel for schedule(static)
        for (long t = 0; t < T; ++t) {
            REAL* dxr = dx + t * K;
            for (long k = 0; k < K; ++k) dxr[k] = 0;
            for (long n = 0; n < N; ++n) {
                REAL g = dout[t * N + n];
                const REAL* wr = W + n * K;
#pragma omp simd
                for (long k = 0; k < K; ++k) dxr[k] += g * wr[k];
            }
        }
    }
    if (dW) {
#pragma omp parallel for schedule(static)
        for (long n = 0; n < N; ++n) {
            REAL* dwr = dW + n * K;
            for (long k = 0; k < K; ++k) dwr[k] = 0;
            for (long t = 0; t < T; ++t) {
                REAL g = dout[t * N + n];
                const REAL* xr = x + t * K;
#pragma omp simd
                for (long k = 0; k < K; ++k) dwr[k] += g * xr[k];
            }
        }
    }
    if (db) {
#pragma omp parallel for schedule(static)
        for (long n = 0; n < N; ++n) {
            REAL s = 0;
            for (long t = 0; t < T; ++t) s += dout[t * N + n];
            db[n] = s;
        }
    }
}

/* ---- GeLU ---- */
/* erf form: gelu(u) = u/2 (1 + erf(u/sqrt2)); gelu'(u) = (1+erf(u/sqrt2))/2 + u exp(-u^2/2)/sqrt(2 pi)
 * tanh form: gelu(u) = u/2 (1 + tanh(c (u + 0.044715 u^3))), c = sqrt(2/pi)                            */
static REAL gelu_val(REAL u, int act)
{
    double x = (double)u;
    if (act == PWO_ACT_GELU_TANH) {
        double c = sqrt(2.0 / M_PI);
        return (REAL)(0.5 * x * (1.0 + tanh(c * (x + 0.044715 * x * x * x))));
    }
    return (REAL)(0.5 * x * (1.0 + erf(x / sqrt(2.0))));
}
static REAL gelu_grad(REAL u, int act)
{
    double x = (double)u;
    if (act == PWO_ACT_GELU_TANH) {
        double c = sqrt(2.0 / M_PI);
        double z = c * (x + 0.044715 * x * x * x);
        double th = tanh(z);
        double dz = c * (1.0 + 3.0 * 0.044715 * x * x);
        return (REAL)(0.5 * (1.0 + th) + 0.5 * x * (1.0 - th * th) * dz);
    }
    return (REAL)(0.5 * (1.0 + erf(x / sqrt(2.0))) + x * exp(-0.5 * x * x) / sqrt(2.0 * M_PI));
}
void FN(pwo_gelu_fwd)(const REAL* u, long n, int act, REAL* a)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) a[i] = gelu_val(u[i], act);
}
void FN(pwo_gelu_bwd)(const REAL* u, const REAL* da, long n, int act, REAL* du)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) du[i] = da[i] * gelu_grad(u[i], act);
}

/* ---- Causal multi-head self-attention ---- */
/* For sequence b, head h, query i: s_j = q_i . k_j / sqrt(dh) for j = 0..i only,
 * p = softmax(s), o_i = sum_j p_j v_j, lse_i = max + log(sum exp(s - max)).
 * Keys j > i are skipped, never multiplied by zero.  probs (may be NULL) receives
 * the full [B,H,S,S] probability tensor with zeros above the diagonal.          */
void FN(pwo_attn_fwd)(const REAL* qkv, long B, long S, long H, long dh, REAL* o, REAL* lse, REAL* probs)
{
    const long d = H * dh, ld = 3 * d;
    const REAL scale = (REAL)(1.0 / sqrt((double)dh));
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long bh = 0; bh < B * H; ++bh)
        for (long i = 0; i < S; ++i) {
            long b = bh / H, h = bh % H;
            REAL* s = (REAL*)malloc((size_t)(i + 1) * sizeof(REAL));
            const REAL* q = qkv + (b * S + i) * ld + h * dh;
            REAL m = -INFINITY;
            for (long j = 0; j <= i; ++j) {
                const REAL* k = qkv + (b * S + j) * ld + d + h * dh;
                REAL acc = 0;
#pragma omp simd reduction(+ : acc)
                for (long c = 0; c < dh; ++c) acc += q[c] * k[c];
                s[j] = acc * scale;
                if (s[j] > m) m = s[j];
            }
            REAL z = 0;
            for (long j = 0; j <= i; ++j) {
                s[j] = (REAL)exp((double)(s[j] - m));
                z += s[j];
            }
            REAL* orow = o + (b * S + i) * d + h * dh;
            for (long c = 0; c < dh; ++c) orow[c] = 0;
            for (long j = 0; j <= i; ++j) {
                REAL p = s[j] / z;
                const REAL* v = qkv + (b * S + j) * ld + 2 * d + h * dh;
                for (long c = 0; c < dh; ++c) orow[c] += p * v[c];
                if (probs) probs[((b * H + h) * S + i) * S + j] = p;
            }
            if (probs)
                for (long j = i + 1; j < S; ++j) probs[((b * H + h) * S + i) * S + j] = 0;
            if (lse) lse[(b * H + h) * S + i] = m + (REAL)log((double)z);
            free(s);
        }
}

/* Backward of causal attention.  p is recomputed from q and k by the definition.
 *   dv_j = sum_{i>=j} p_ij do_i          dp_ij = do_i . v_j
 *   ds_ij = p_ij (dp_ij - sum_j' p_ij' dp_ij')
 *   dq_i = (1/sqrt dh) sum_{j<=i} ds_ij k_j     dk_j = (1/sqrt dh) sum_{i>=j} ds_ij q_i
 * One thread owns one (b,h), so the sums over i into dk/dv need no atomics.      */
void FN(pwo_attn_bwd)(const REAL* qkv, const REAL* dout, long B, long S, long H, long dh, REAL* dqkv)
{
    const long d = H * dh, ld = 3 * d;
    const REAL scale = (REAL)(1.0 / sqrt((double)dh));
#pragma omp parallel for schedule(dynamic, 1)
    for (long bh = 0; bh < B * H; ++bh) {
        long b = bh / H, h = bh % H;
        REAL* p = (REAL*)malloc((size_t)S * sizeof(REAL));
        REAL* dp = (REAL*)malloc((size_t)S * sizeof(REAL));
        for (long i = 0; i < S; ++i)
            for (long part = 0; part < 3; ++part) {
                REAL* g = dqkv + (b * S + i) * ld + part * d + h * dh;
                for (long c = 0; c < dh; ++c) g[c] = 0;
            }
        for (long i = 0; i < S; ++i) {
            const REAL* q = qkv + (b * S + i) * ld + h * dh;
            const REAL* go = dout + (b * S + i) * d + h * dh;
            REAL m = -INFINITY;
            for (long j = 0; j <= i; ++j) {
                const REAL* k = qkv + (b * S + j) * ld + d + h * dh;
                REAL acc = 0;
#pragma omp simd reduction(+ : acc)
                for (long c = 0; c < dh; ++c) acc += q[c] * k[c];
                p[j] = acc * scale;
                if (p[j] > m) m = p[j];
            }
            REAL z = 0;
            for (long j = 0; j <= i; ++j) {
                p[j] = (REAL)exp((double)(p[j] - m));
                z += p[j];
            }
            REAL dot = 0;
            for (long j = 0; j <= i; ++j) {
                p[j] /= z;
                const REAL* v = qkv + (b * S + j) * ld + 2 * d + h * dh;
                REAL acc = 0;
#pragma omp simd reduction(+ : acc)
                for (long c = 0; c < dh; ++c) acc += go[c] * v[c];
                dp[j] = acc;
                dot += p[j] * acc;
            }
            REAL* dq = dqkv + (b * S + i) * ld + h * dh;
            for (long j = 0; j <= i; ++j) {
                REAL ds = p[j] * (dp[j] - dot);
                const REAL* k = qkv + (b * S + j) * ld + d + h * dh;
                REAL* dk = dqkv + (b * S + j) * ld + d + h * dh;
                REAL* dv = dqkv + (b * S + j) * ld + 2 * d + h * dh;
                for (long c = 0; c < dh; ++c) {
                    dq[c] += scale * ds * k[c];
                    dk[c] += scale * ds * q[c];
                    dv[c] += p[j] * go[c];
                }
            }
        }
        free(p);
        free(dp);
    }
}

/* ---- One pre-LN decoder layer ---- */
/* params[12]: ln1_gamma[d] ln1_beta[d] w_qkv[3d,d] b_qkv[3d] w_o[d,d] b_o[d]
 *             ln2_gamma[d] ln2_beta[d] w_fc1[F,d] b_fc1[F] w_fc2[d,F] b_fc2[d]
 * saved[12]:  h1[T,d] qkv[T,3d] o[T,d] x1[T,d] h2[T,d] u[T,F] a[T,F] lse[B,H,S]
 *             mu1[T] r1[T] mu2[T] r2[T]      (all written by the forward)
 *   x1 = x + attn(LN1(x)) Wo^T + bo ;  y = x1 + gelu(LN2(x1) W1^T + b1) W2^T + b2   */
enum { P_G1, P_B1, P_WQKV, P_BQKV, P_WO, P_BO, P_G2, P_B2, P_W1, P_BF1, P_W2, P_BF2 };
enum { S_H1, S_QKV, S_O, S_X1, S_H2, S_U, S_A, S_LSE, S_MU1, S_R1, S_MU2, S_R2 };

void FN(pwo_layer_fwd)(long B, long S, long d, long H, long dh, long F, double eps, int act,
                       const REAL* const* params, const REAL* x, REAL* const* saved, REAL* y)
{
    const long T = B * S;
    FN(pwo_ln_fwd)(x, params[P_G1], params[P_B1], T, d, eps, saved[S_H1], saved[S_MU1], saved[S_R1]);
    FN(pwo_linear_fwd)(saved[S_H1], params[P_WQKV], params[P_BQKV], T, d, 3 * d, saved[S_QKV]);
    FN(pwo_attn_fwd)(saved[S_QKV], B, S, H, dh, saved[S_O], saved[S_LSE], NULL);
    FN(pwo_linear_fwd)(saved[S_O], params[P_WO], params[P_BO], T, d, d, saved[S_X1]);
    for (long i = 0; i < T * d; ++i) saved[S_X1][i] += x[i];
    FN(pwo_ln_fwd)(saved[S_X1], params[P_G2], params[P_B2], T, d, eps, saved[S_H2], saved[S_MU2], saved[S_R2]);
    FN(pwo_linear_fwd)(saved[S_H2], params[P_W1], params[P_BF1], T, d, F, saved[S_U]);
    FN(pwo_gelu_fwd)(saved[S_U], T * F, act, saved[S_A]);
    FN(pwo_linear_fwd)(saved[S_A], params[P_W2], params[P_BF2], T, F, d, y);
    for (long i = 0; i < T * d; ++i) y[i] += saved[S_X1][i];
}

/* Backward of the layer given dy.  grads[12] are shaped like params; with
 * accumulate != 0 the new gradients are added to what grads already hold
 * (sum over micro-batches, no averaging), otherwise they overwrite.            */
static void add_or_set(REAL* dst, const REAL* src, long n, int accumulate)
{
    for (long i = 0; i < n; ++i) dst[i] = accumulate ? dst[i] + src[i] : src[i];
}

void FN(pwo_layer_bwd)(long B, long S, long d, long H, long dh, long F, int act,
                       const REAL* const* params, const REAL* x, const REAL* const* saved,
                       const REAL* dy, REAL* dx, REAL* const* grads, int accumulate)
{
    const long T = B * S;
    (void)dh;
    REAL* da = (REAL*)malloc((size_t)(T * F) * sizeof(REAL));
    REAL* du = (REAL*)malloc((size_t)(T * F) * sizeof(REAL));
    REAL* dh2 = (REAL*)malloc((size_t)(T * d) * sizeof(REAL));
    REAL* dx1 = (REAL*)malloc((size_t)(T * d) * sizeof(REAL));
    REAL* dob = (REAL*)malloc((size_t)(T * d) * sizeof(REAL));
    REAL* dqkv = (REAL*)malloc((size_t)(T * 3 * d) * sizeof(REAL));
    REAL* dh1 = (REAL*)malloc((size_t)(T * d) * sizeof(REAL));
    const long wmax = (3 * d * d > d * F) ? 3 * d * d : d * F;
    REAL* gw = (REAL*)malloc((size_t)wmax * sizeof(REAL));
    REAL* gb = (REAL*)malloc((size_t)((F > 3 * d ? F : 3 * d)) * sizeof(REAL));
    REAL* gb2 = (REAL*)malloc((size_t)d * sizeof(REAL));

    /* y = x1 + a W2^T + b2 */
    FN(pwo_linear_bwd)(saved[S_A], params[P_W2], dy, T, F, d, da, gw, gb);
    add_or_set(grads[P_W2], gw, d * F, accumulate);
    add_or_set(grads[P_BF2], gb, d, accumulate);
    /* a = gelu(u) */
    FN(pwo_gelu_bwd)(saved[S_U], da, T * F, act, du);
    /* u = h2 W1^T + b1 */
    FN(pwo_linear_bwd)(saved[S_H2], params[P_W1], du, T, d, F, dh2, gw, gb);
    add_or_set(grads[P_W1], gw, F * d, accumulate);
    add_or_set(grads[P_BF1], gb, F, accumulate);
    /* h2 = LN2(x1); x1 also feeds the residual */
    FN(pwo_ln_bwd)(dh2, saved[S_X1], saved[S_MU2], saved[S_R2], params[P_G2], T, d, dx1, gb, gb2);
    add_or_set(grads[P_G2], gb, d, accumulate);
    add_or_set(grads[P_B2], gb2, d, accumulate);
    for (long i = 0; i < T * d; ++i) dx1[i] += dy[i];
    /* x1 = x + o Wo^T + bo */
    FN(pwo_linear_bwd)(saved[S_O], params[P_WO], dx1, T, d, d, dob, gw, gb);
    add_or_set(grads[P_WO], gw, d * d, accumulate);
    add_or_set(grads[P_BO], gb, d, accumulate);
    /* o = attention(qkv) */
    FN(pwo_attn_bwd)(saved[S_QKV], dob, B, S, H, d / H, dqkv);
    /* qkv = h1 Wqkv^T + bqkv */
    FN(pwo_linear_bwd)(saved[S_H1], params[P_WQKV], dqkv, T, d, 3 * d, dh1, gw, gb);
    add_or_set(grads[P_WQKV], gw, 3 * d * d, accumulate);
    add_or_set(grads[P_BQKV], gb, 3 * d, accumulate);
    /* h1 = LN1(x); x also feeds the residual */
    FN(pwo_ln_bwd)(dh1, x, saved[S_MU1], saved[S_R1], params[P_G1], T, d, dx, gb, gb2);
    add_or_set(grads[P_G1], gb, d, accumulate);
    add_or_set(grads[P_B1], gb2, d, accumulate);
    for (long i = 0; i < T * d; ++i) dx[i] += dx1[i];

    free(da); free(du); free(dh2); free(dx1); free(dob); free(dqkv); free(dh1);
    free(gw); free(gb); free(gb2);
}

/* ---- First and last layer of the language model (Section 5.3 names an embedding layer first and a
 * softmax layer last).  The paper gives no formula; these are the textbook ones, with the
 * output projection tied to the embedding table (reading listed in the design notes). ---- */

/* Embedding lookup: x0[t][:] = E[ids[t]][:]. */
void FN(pwo_embed_fwd)(const int* ids, const REAL* E, long T, long d, REAL* x0)
{
    for (long t = 0; t < T; ++t)
        for (long c = 0; c < d; ++c) x0[t * d + c] = E[(long)ids[t] * d + c];
}

/* Backward of the lookup: dE[ids[t]][:] += dx0[t][:], tokens visited in order. */
void FN(pwo_embed_bwd)(const int* ids, const REAL* dx0, long T, long d, REAL* dE)
{
    for (long t = 0; t < T; ++t)
        for (long c = 0; c < d; ++c) dE[(long)ids[t] * d + c] += dx0[t * d + c];
}

/* Tied softmax head with cross-entropy against integer labels:
 *   z[t][v] = sum_c hf[t][c] E[v][c]
 *   lse[t]  = log sum_v exp(z[t][v])          (computed as max + log sum exp(z - max))
 *   loss    = (1/T) sum_t ( lse[t] - z[t][label[t]] )
 * logits (may be NULL) receives z. */
void FN(pwo_head_fwd)(const REAL* hf, const REAL* E, const int* labels, long T, long d, long V,
                      REAL* logits, REAL* lse, REAL* loss)
{
    double total = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : total)
    for (long t = 0; t < T; ++t) {
        REAL* z = (REAL*)malloc(sizeof(REAL) * (size_t)V);
        REAL mx = -INFINITY;
        for (long v = 0; v < V; ++v) {
            REAL acc = 0;
            for (long c = 0; c < d; ++c) acc += hf[t * d + c] * E[v * d + c];
            z[v] = acc;
            if (acc > mx) mx = acc;
        }
        double sum = 0.0;
        for (long v = 0; v < V; ++v) sum += exp((double)(z[v] - mx));
        const double l = (double)mx + log(sum);
        lse[t] = (REAL)l;
        total += l - (double)z[labels[t]];
        if (logits) for (long v = 0; v < V; ++v) logits[t * V + v] = z[v];
        free(z);
    }
    *loss = (REAL)(total / (double)T);
}

/* Backward of the head for d loss = 1:
 *   dz[t][v]  = ( exp(z[t][v] - lse[t]) - [v == label[t]] ) / T
 *   dhf[t][c] = sum_v dz[t][v] E[v][c]
 *   dE[v][c] += sum_t dz[t][v] hf[t][c]
 * dlogits (may be NULL) receives dz.  z is recomputed from hf and E by the definition. */
void FN(pwo_head_bwd)(const REAL* hf, const REAL* E, const int* labels, const REAL* lse, long T, long d, long V,
                      REAL* dhf, REAL* dE, REAL* dlogits)
{
    REAL* dz = (REAL*)malloc(sizeof(REAL) * (size_t)T * (size_t)V);
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        for (long v = 0; v < V; ++v) {
            REAL acc = 0;
            for (long c = 0; c < d; ++c) acc += hf[t * d + c] * E[v * d + c];
            REAL g = (REAL)exp((double)(acc - lse[t]));
            if (v == (long)labels[t]) g -= (REAL)1;
            dz[t * V + v] = g / (REAL)T;
        }
        for (long c = 0; c < d; ++c) {
            REAL acc = 0;
            for (long v = 0; v < V; ++v) acc += dz[t * V + v] * E[v * d + c];
            dhf[t * d + c] = acc;
        }
    }
#pragma omp parallel for schedule(static)
    for (long v = 0; v < V; ++v)
        for (long c = 0; c < d; ++c) {
            REAL acc = 0;
            for (long t = 0; t < T; ++t) acc += dz[t * V + v] * hf[t * d + c];
            dE[v * d + c] += acc;
        }
    if (dlogits) memcpy(dlogits, dz, sizeof(REAL) * (size_t)T * (size_t)V);
    free(dz);
}

/* ---- The three one-line computations of the paper's Figure 2 program are all of the form
 * y = x * scale + shift (a: x*2, b: x+1, c: x/2). ---- */
void FN(pwo_affine)(const REAL* x, long n, double scale, double shift, REAL* y)
{
    for (long i = 0; i < n; ++i) y[i] = (REAL)((double)x[i] * scale + shift);
}


/* ---- Gradient apply ----
 * In the appendix's trace of data-parallel training over two islands, each island applies
 * the gradients it received before it starts the next step.  The paper names no optimizer,
 * so this is plain stochastic gradient descent on a full-precision master copy of a
 * parameter tensor, with the bf16 working copy derived from the master afterwards:
 *     master <- master - lr * grad_scale * grad          (grad_scale: e.g. 1 / micro-batches)
 *     param  =  master rounded to bf16 (8 significant bits, round to nearest, ties to even)
 * The rounding is the definition written out: split x = m * 2^e with 0.5 <= |m| < 1, round
 * m * 2^8 to the nearest integer (ties to even: the default rounding mode of nearbyint) and
 * scale back.  Values below the bf16 normal range do not occur in this workload. */
REAL FN(pwo_round_bf16)(REAL x)
{
    if (x == 0 || !isfinite((double)x)) return x;
    int e;
    const double m = frexp((double)x, &e);
    return (REAL)ldexp(nearbyint(ldexp(m, 8)), e - 8);
}

void FN(pwo_sgd_apply)(REAL* master, const REAL* grad, long n, double lr, double grad_scale, REAL* param)
{
    for (long i = 0; i < n; ++i) {
        master[i] = (REAL)((double)master[i] - lr * grad_scale * (double)grad[i]);
        param[i] = FN(pwo_round_bf16)(master[i]);
    }
}
