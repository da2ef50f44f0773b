/*
 * pw.h - C ABI of the B200 (sm_100a) decoder-layer engine.
 *
 * The Pathways paper (arXiv 2203.12533) schedules "compiled functions": sub-computations
 * with static shapes whose resource needs are known before they run (Section 3; Appendix B),
 * enqueued asynchronously on an accelerator with buffer futures as inputs (Sections 4.4-4.5).
 * For its decoder-only language-model workload (Section 5.3: 62 layers, model dimension 2048,
 * hidden dimension 8192, micro-batches of 4 examples, GPipe-like schedule) the compiled
 * function a pipeline stage runs is a stack of Transformer layers, forward and backward, on
 * one micro-batch.  This library is that function for one GPU:
 *
 *   pw_layer_create / pw_layer_fwd / pw_layer_bwd    one pre-LN causal decoder layer
 *   pw_stage_create / pw_stage_run_chain             a stack of layers over M micro-batches
 *
 * Conventions shared by every call
 *   - All tensor pointers are DEVICE pointers unless a parameter is documented as host.
 *     Activations are bf16, row-major [B, S, width] (token t = b*S + s).  Weights are bf16,
 *     row-major [out_features, in_features] (y = x W^T + b).  Parameter gradients are fp32
 *     with the shape of the parameter.  LayerNorm statistics and log-sum-exp are fp32.
 *   - Ownership: the caller owns every device buffer it passes and keeps it alive until the
 *     stream has passed the enqueued work.  The library owns only host-side handles, one
 *     small device status word per handle, and cached CUDA graphs.  No call on the enqueue
 *     path allocates device memory.
 *   - Asynchrony: fwd / bwd / run_chain only enqueue work on `stream` (a cudaStream_t passed
 *     as void*; NULL = the legacy default stream) and return without synchronising - stream
 *     order plays the role of the paper's buffer futures.  Argument errors are detected
 *     before anything is enqueued.
 *   - Errors: every call returns a pw_status_t; no exception crosses the boundary.
 *     pw_last_error() gives a thread-local message for the last failure on this thread.
 *     Device-side waits are bounded: if one expires the kernel records PW_ERR_TIMEOUT in the
 *     handle's status word, releases what it holds and returns; pw_layer_status /
 *     pw_stage_status read that word.
 *   - Threading: a handle is used by one host thread at a time.
 *   - Device: compute capability 10.x only; there is no fallback path of any kind.
 *
 * Arithmetic (the paper gives sizes only; these are the textbook definitions)
 *   h1 = LN(x; g1, b1)                 qkv = h1 Wqkv^T + bqkv      (columns: q | k | v, head h at h*dh)
 *   o  = causal softmax(q k^T / sqrt(dh)) v   per sequence and head; key j visible to query i iff j <= i
 *   x1 = x + o Wo^T + bo               h2 = LN(x1; g2, b2)
 *   u  = h2 W1^T + b1                  a = GeLU(u)                 y = x1 + a W2^T + b2
 *   LayerNorm: biased variance over the last dimension, eps inside the square root.
 *   bf16 storage, fp32 accumulation / statistics / softmax / GeLU.
 */
#ifndef PW_H_
#define PW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PW_VERSION 100

typedef enum pw_status {
    PW_OK = 0,
    PW_ERR_INVALID_ARG = 1,
    PW_ERR_UNSUPPORTED_SHAPE = 2,
    PW_ERR_WORKSPACE_TOO_SMALL = 3,
    PW_ERR_CUDA = 4,
    PW_ERR_DEVICE_UNSUPPORTED = 5,
    PW_ERR_TIMEOUT = 6,
    PW_ERR_INTERNAL = 7
} pw_status_t;

enum { PW_ACT_GELU_ERF = 0, PW_ACT_GELU_TANH = 1 };
/* Layer flags.  PW_FLAG_LEAN_CTX: the forward does not keep the two LayerNorm outputs (h1, h2) nor
 * GeLU(u) in ctx - 2 T d + T F of the 7 T d + 2 T F bf16 elements a full ctx holds (40 % at
 * F = 4 d).  The backward re-derives them into scratch (two LayerNorm forwards from x and x1 with
 * the same bits as the first time, and GeLU of the bf16 pre-activations u, which may differ from
 * the forward's GeLU of the fp32 pre-activations in the last bf16 bit).  pw_layer_ctx_offset reports
 * size 0 for the three tensors; pw_layer_fwd then needs `scratch` even when ctx is given. */
enum { PW_FLAG_LEAN_CTX = 1u, PW_FLAG_WHOLE_LAYER = 2u };
/* PW_FLAG_WHOLE_LAYER: pw_layer_fwd and pw_layer_bwd are ONE cooperative kernel launch each instead of
 * 7 and 15 - for calls so small that launches and hand-offs between kernels, not arithmetic, set the
 * time (Section 5.1, Figures 5 and 6: computations shorter than the cost of issuing them).  Same
 * tensors, same saved context, same bf16 hand-off points as the default path; results agree with
 * it within rounding (different tile shapes and summation orders), bit-reproducibly.  Supported:
 * head_dim 64, d_model <= 512, seq_len <= 1024, (batch * seq_len / 64) * (d_model / 64) <= 1024; not
 * together with PW_FLAG_LEAN_CTX; pw_layer_fwd needs `scratch` even when ctx is given.  Anything else:
 * PW_ERR_UNSUPPORTED_SHAPE / PW_ERR_INVALID_ARG from pw_layer_create.  A grid barrier that waits
 * longer than about a second records PW_ERR_TIMEOUT in the status word and the kernel returns. */

/* Static shape of a layer call - fixed for the life of the handle, like the static shapes of
 * a compiled function (Section 3).  Supported: head_dim in {64, 128}; n_heads*head_dim ==
 * d_model; d_model % 256 == 0 and d_model <= 8192; d_ff % 128 == 0; seq_len % 128 == 0;
 * batch >= 1; causal == 1.  Anything else gives PW_ERR_UNSUPPORTED_SHAPE (never a slow path). */
typedef struct pw_layer_config {
    uint32_t struct_size; /* sizeof(pw_layer_config_t), for versioning */
    int32_t d_model;
    int32_t n_heads;
    int32_t head_dim;
    int32_t d_ff;
    int32_t seq_len;
    int32_t batch;
    int32_t act;    /* PW_ACT_GELU_ERF (default) or PW_ACT_GELU_TANH */
    float ln_eps;   /* 0 means 1e-5 */
    int32_t causal; /* must be 1 */
    uint32_t flags; /* 0, PW_FLAG_LEAN_CTX or PW_FLAG_WHOLE_LAYER */
} pw_layer_config_t;

/* The 12 parameters of a layer (bf16 device pointers). */
typedef struct pw_layer_params {
    const void* ln1_gamma; /* [d]      */
    const void* ln1_beta;  /* [d]      */
    const void* w_qkv;     /* [3d, d]  */
    const void* b_qkv;     /* [3d]     */
    const void* w_o;       /* [d, d]   */
    const void* b_o;       /* [d]      */
    const void* ln2_gamma; /* [d]      */
    const void* ln2_beta;  /* [d]      */
    const void* w_fc1;     /* [F, d]   */
    const void* b_fc1;     /* [F]      */
    const void* w_fc2;     /* [d, F]   */
    const void* b_fc2;     /* [d]      */
} pw_layer_params_t;

/* Gradients of the 12 parameters (fp32 device pointers, same shapes, same order). */
typedef struct pw_layer_grads {
    void* ln1_gamma; void* ln1_beta; void* w_qkv; void* b_qkv; void* w_o; void* b_o;
    void* ln2_gamma; void* ln2_beta; void* w_fc1; void* b_fc1; void* w_fc2; void* b_fc2;
} pw_layer_grads_t;

typedef struct pw_layer pw_layer_t;
typedef struct pw_stage pw_stage_t;

/* Tensors the forward saves in `ctx` for the backward (ids for pw_layer_ctx_offset). */
enum {
    PW_CTX_H1 = 0,  /* bf16 [T, d]   LN1 output              */
    PW_CTX_QKV = 1, /* bf16 [T, 3d]                          */
    PW_CTX_O = 2,   /* bf16 [T, d]   attention output        */
    PW_CTX_X1 = 3,  /* bf16 [T, d]   x + attention branch    */
    PW_CTX_H2 = 4,  /* bf16 [T, d]   LN2 output              */
    PW_CTX_U = 5,   /* bf16 [T, F]   FC1 pre-activation      */
    PW_CTX_A = 6,   /* bf16 [T, F]   GeLU(u)                 */
    PW_CTX_LSE = 7, /* fp32 [B, H, S] log-sum-exp of the scaled, masked scores */
    PW_CTX_MU1 = 8, PW_CTX_R1 = 9,   /* fp32 [T] LN1 mean and 1/sqrt(var+eps) */
    PW_CTX_MU2 = 10, PW_CTX_R2 = 11, /* fp32 [T] LN2 */
    PW_CTX_COUNT = 12
};

/* ---- misc ---- */
int pw_version(void);
const char* pw_status_string(pw_status_t s);
/* Thread-local description of the last error returned on this thread ("" if none). */
const char* pw_last_error(void);

/* ---- one layer (Section 5.3's Transformer layer as a compiled function, Section 3) ---- */

/* Validates cfg, checks the current device (PW_ERR_DEVICE_UNSUPPORTED unless sm_100), builds
 * the static launch plan.  *out is set only on PW_OK.  Host pointers. */
pw_status_t pw_layer_create(const pw_layer_config_t* cfg, pw_layer_t** out);
void pw_layer_destroy(pw_layer_t* layer);

/* Bytes the caller must provide: ctx (saved activations, written by fwd and read by bwd) and
 * scratch (temporaries of one fwd or bwd call; contents are undefined between calls).
 * Both must be 256-byte aligned device memory.  Host pointers for the outputs. */
pw_status_t pw_layer_workspace_bytes(const pw_layer_t* layer, size_t* ctx_bytes, size_t* scratch_bytes);

/* Where tensor `which` (PW_CTX_*) lives inside ctx: byte offset and size.  For tests/tools. */
pw_status_t pw_layer_ctx_offset(const pw_layer_t* layer, int which, size_t* offset, size_t* bytes);

/* y = layer(x).  x, y: bf16 [B,S,d] device, y must not alias x.  ctx: receives the saved
 * activations; NULL means "save nothing" (the intermediates then live in scratch only).
 * scratch may be NULL only if ctx is given and the layer is not PW_FLAG_LEAN_CTX.
 * `params` is a host struct of device pointers.  Enqueue only. */
pw_status_t pw_layer_fwd(pw_layer_t* layer, const pw_layer_params_t* params, const void* x, void* y,
                         void* ctx, void* scratch, void* stream);

/* dx and parameter gradients from dy.  dy, dx: bf16 [B,S,d] device; dx may alias dy.
 * accumulate = 0: gradients overwrite *grads; 1: they are added (sum over micro-batches, no
 * averaging).  ctx: what fwd wrote for the same x and params; NULL means recompute: the
 * forward is re-run from x into scratch first (bit-identical to the first forward), then the
 * backward runs.  `grads` is a host struct of device pointers.  Enqueue only. */
pw_status_t pw_layer_bwd(pw_layer_t* layer, const pw_layer_params_t* params, const void* x, const void* dy,
                         void* dx, const pw_layer_grads_t* grads, int accumulate, const void* ctx,
                         void* scratch, void* stream);

/* Synchronises the device and reads the handle's status word: *device_status = PW_OK or the
 * code a kernel recorded (PW_ERR_TIMEOUT) with *site (may be NULL) = where it gave up. */
pw_status_t pw_layer_status(pw_layer_t* layer, int* device_status, int* site);

/* Per-kernel timing for benchmarks.  Between profile_begin and profile_end every kernel this
 * handle launches is bracketed by CUDA events on the launching stream; profile_end synchronises
 * that stream and sums the elapsed times by kernel class.  Not usable inside a captured graph
 * (PW_DISPATCH_GRAPH returns PW_ERR_INVALID_ARG while profiling is on).  Host structs. */
enum {
    PW_K_GEMM_TN = 0,   /* forward GEMMs                      */
    PW_K_GEMM_NN = 1,   /* data-gradient GEMMs                */
    PW_K_GEMM_NT = 2,   /* weight-gradient GEMMs              */
    PW_K_ATTN_FWD = 3,
    PW_K_ATTN_BWD = 4,  /* delta + dq + dkdv kernels          */
    PW_K_LN_FWD = 5,
    PW_K_LN_BWD = 6,    /* main kernel (+ partial reduction when called as a single step) */
    PW_K_COLSUM = 7,    /* main kernel (+ partial reduction when called as a single step) */
    PW_K_XENT = 8,      /* softmax / cross-entropy + loss mean (pw_lm_step)          */
    PW_K_EMBED = 9,     /* embedding lookup and its scatter-add backward (pw_lm_step) */
    PW_K_GELU = 10,     /* GeLU(u) re-derived in the backward of a PW_FLAG_LEAN_CTX layer */
    PW_K_WHOLE_LAYER = 11, /* forward or backward of a PW_FLAG_WHOLE_LAYER handle (one launch each) */
    PW_K_REDUCE = 12,   /* one launch per layer backward: fixed-order sums of the partial rows that its two
                           LayerNorm backward kernels and its two bias column sums left (8 gradient vectors) */
    PW_K_COUNT = 13
};
typedef struct pw_profile {
    uint64_t launches[PW_K_COUNT]; /* kernel launches per class since profile_begin      */
    double ms[PW_K_COUNT];         /* summed device time per class, milliseconds         */
    double flops[PW_K_COUNT];      /* executed tensor-core FLOPs (GEMM / attention classes; causal half only) */
    double bytes[PW_K_COUNT];      /* algorithmic HBM bytes (LN / column-sum classes)    */
} pw_profile_t;
pw_status_t pw_layer_profile_begin(pw_layer_t* layer);
pw_status_t pw_layer_profile_end(pw_layer_t* layer, pw_profile_t* out);
/* Kernels launched through this handle since it was created (graph replays count their nodes). */
pw_status_t pw_layer_launch_count(const pw_layer_t* layer, uint64_t* count);
/* The backward pass runs its weight-gradient GEMMs and bias column sums on a library-owned side
 * stream beside the data-gradient chain (default).  enabled = 0 keeps every kernel on the calling
 * stream, in program order - the same kernels, the same results, one after the other: what a
 * per-kernel time measured alone corresponds to.  Takes effect from the next call. */
pw_status_t pw_layer_set_side_stream(pw_layer_t* layer, int enabled);

/* ---- a pipeline stage: L layers x M micro-batches (Section 5.3, Table 2; dispatch modes of Section 5.1) ---- */

enum {
    PW_DISPATCH_OPBYOP = 0, /* synchronise the stream after every layer call (the paper's OpByOp) */
    PW_DISPATCH_ASYNC = 1,  /* enqueue the whole chain, return (the paper's Chained)             */
    PW_DISPATCH_GRAPH = 2   /* capture the chain once into a CUDA graph, replay it (Fused)       */
};
enum {
    PW_SCHEDULE_GPIPE = 0,         /* all M forwards, then all M backwards (GPipe-like, Section 5.3) */
    PW_SCHEDULE_PER_MICROBATCH = 1 /* forward and backward of micro-batch m before m+1              */
};

pw_status_t pw_stage_create(const pw_layer_config_t* cfg, int n_layers, pw_stage_t** out);
void pw_stage_destroy(pw_stage_t* stage);

/* Workspace (device, 256-byte aligned) needed by pw_stage_run_chain for these settings. */
pw_status_t pw_stage_workspace_bytes(const pw_stage_t* stage, int n_microbatches, int schedule, int recompute,
                                     size_t* bytes);

/* For each micro-batch m: x_mb[m] -> L layers -> y_mb[m]; dy_mb[m] -> L layers backward ->
 * dx_mb[m].  Layer l+1 consumes layer l's bf16 output.  grads[l] receive the SUM over the M
 * micro-batches (overwritten by micro-batch 0, added to by the rest).
 *   params, grads : host arrays [L] of structs of device pointers
 *   x_mb, dy_mb, y_mb, dx_mb : host arrays [M] of device pointers (bf16 [B,S,d] each);
 *                   y_mb[m] must not alias x_mb[m]
 *   recompute = 1 : only each layer's input is kept for the backward; the layer's forward is
 *                   re-run inside its backward (the pipeline-stage workload after Section 5.3 runs this way)
 *   recompute = 0 : every layer saves its activations (needs L * M (GPipe) or L (per-micro-batch)
 *                   contexts in the workspace)
 * GRAPH mode caches an instantiated graph keyed by every pointer and setting of the call and
 * replays it when they repeat.  Returns PW_ERR_WORKSPACE_TOO_SMALL before enqueuing anything
 * if workspace_bytes is insufficient.  Enqueue only (OPBYOP synchronises by definition). */
pw_status_t pw_stage_run_chain(pw_stage_t* stage, const pw_layer_params_t* params, const pw_layer_grads_t* grads,
                               const void* const* x_mb, const void* const* dy_mb, void* const* y_mb,
                               void* const* dx_mb, int n_microbatches, int dispatch_mode, int schedule,
                               int recompute, void* workspace, size_t workspace_bytes, void* stream);

pw_status_t pw_stage_status(pw_stage_t* stage, int* device_status, int* site);
pw_status_t pw_stage_profile_begin(pw_stage_t* stage);
pw_status_t pw_stage_profile_end(pw_stage_t* stage, pw_profile_t* out);
pw_status_t pw_stage_launch_count(const pw_stage_t* stage, uint64_t* count);
pw_status_t pw_stage_set_side_stream(pw_stage_t* stage, int enabled);   /* as pw_layer_set_side_stream */

/* ---- the whole small language model: embedding layer first, softmax layer last (Section 5.3) ----
 * The paper names the two end layers but prints no formula; the reading built here: token
 * embedding E [V,d] (no positional term), L decoder layers, a final LayerNorm, logits = hf E^T with
 * the SAME table (tied), loss = mean over the T tokens of -log softmax(logits)[label].
 *   ids, labels : int32 [B,S] device, values in [0, vocab) (anything else is reported through the
 *                 status word as PW_ERR_INVALID_ARG and treated as 0)
 *   loss        : one fp32 on the device
 *   gradients   : overwritten (one batch per call): per-layer grads as in pw_layer_bwd,
 *                 lm_grads->embedding fp32 [V,d] = head part + scatter-add of the input gradient
 *                 (tokens added in increasing order: bitwise reproducible), lnf_gamma / lnf_beta fp32 [d]
 * vocab % 8 == 0.  The logits (bf16 [T,V]) live in the workspace and are turned into their own
 * gradient in place.  Enqueue only. */
typedef struct pw_lm_params {
    const void* embedding; /* bf16 [V, d]; also the output projection */
    const void* lnf_gamma; /* bf16 [d] final LayerNorm */
    const void* lnf_beta;  /* bf16 [d] */
} pw_lm_params_t;
typedef struct pw_lm_grads {
    void* embedding; /* fp32 [V, d] */
    void* lnf_gamma; /* fp32 [d] */
    void* lnf_beta;  /* fp32 [d] */
} pw_lm_grads_t;
pw_status_t pw_lm_workspace_bytes(const pw_stage_t* stage, int vocab, int recompute, size_t* bytes);
pw_status_t pw_lm_step(pw_stage_t* stage, const pw_layer_params_t* params, const pw_layer_grads_t* grads,
                       const pw_lm_params_t* lm, const pw_lm_grads_t* lm_grads, const int32_t* ids,
                       const int32_t* labels, float* loss, int vocab, int recompute, void* workspace,
                       size_t workspace_bytes, void* stream);

/* ---- single steps of the layer (same kernels the layer calls; for unit tests and profiling) ---- */

/* LayerNorm forward.  x,h: bf16 [T,d]; gamma,beta: bf16 [d]; mu,rstd: fp32 [T]. */
pw_status_t pw_op_layernorm_fwd(const void* x, const void* gamma, const void* beta, int T, int d, float eps,
                                void* h, void* mu, void* rstd, void* stream);

/* LayerNorm backward fused with the residual-gradient add and two bias-gradient column sums:
 *   dx = resid + LNbwd(dh; x, mu, rstd, gamma)          (bf16 [T,d]; resid bf16 [T,d])
 *   dgamma, dbeta (fp32 [d])  (+)= sum_t dh*xhat, sum_t dh
 *   db_resid (fp32 [d], may be NULL) (+)= sum_t resid ; db_dx (fp32 [d], may be NULL) (+)= sum_t dx
 * partials: fp32 device scratch of pw_op_layernorm_bwd_scratch_bytes(T, d) bytes. */
size_t pw_op_layernorm_bwd_scratch_bytes(int T, int d);
pw_status_t pw_op_layernorm_bwd(const void* dh, const void* x, const void* mu, const void* rstd,
                                const void* gamma, const void* resid, int T, int d, void* dx, void* dgamma,
                                void* dbeta, void* db_resid, void* db_dx, int accumulate, void* partials,
                                void* stream);

/* Column sums: out[n] (+)= sum_t in[t][n]; in bf16 [T,N] (row stride ld elements), out fp32 [N].
 * partials: fp32 device scratch of pw_op_colsum_scratch_bytes(T, N) bytes. */
size_t pw_op_colsum_scratch_bytes(int T, int N);
pw_status_t pw_op_colsum(const void* in, int T, int N, int ld, void* out, int accumulate, void* partials,
                         void* stream);

/* Column sums for callers that cannot allocate device memory (the paper has no counterpart; this
 * is a convenience of this library).  Same result as pw_op_colsum up to summation order, but the
 * partial sums live in a 1 MiB array built into the library instead of a caller buffer, and the
 * call itself allocates nothing on host-visible CUDA APIs: no cudaMalloc / cudaFree, no
 * allocating library routine.  It is meant for code that runs when allocation is off the table:
 * a serving loop whose memory pools already own all of HBM, a host callback, a plugin that is
 * handed buffers but no allocator.
 *   in  bf16 [T, N] device (row stride ld elements, ld >= N); out fp32 [N] device;
 *   accumulate 0: out = sums, 1: out += sums.  N % 8 == 0, ld % 8 == 0.
 * Limit: N <= 262144 columns (the array holds 262144 floats); beyond it the call returns
 * PW_ERR_WORKSPACE_TOO_SMALL and launches nothing.  Fewer row groups are used than in
 * pw_op_colsum when N is large, so the two may differ in the last fp32 bits.
 * The first call on a device looks up the array's device address (once per device, with that
 * device current); make that first call outside any stream capture.  Every call on a device
 * shares the one array, which keeps the previous call's partial sums (each call overwrites the
 * slots it later reads, so nothing needs clearing); calls whose kernels overlap on the GPU -
 * different streams, or graphs replayed concurrently - race on it and must be serialised by the
 * caller.  Each GPU that loads the library holds the 1 MiB until the process exits. */
pw_status_t pw_op_colsum_noalloc(const void* in, int T, int N, int ld, void* out, int accumulate, void* stream);

/* bf16 GEMM on the tensor cores, fp32 accumulation.  C[M,N] = op(A) op(B) then an epilogue.
 *   layout PW_GEMM_TN: A is [M,K] row-major (lda), B is [N,K] row-major (ldb)      (forward:  x W^T)
 *          PW_GEMM_NN: A is [M,K] row-major,       B is [K,N] row-major            (dgrad:    dy W)
 *          PW_GEMM_NT: A is [K,M] row-major,       B is [K,N] row-major            (wgrad:    dy^T x)
 *   epilogue PW_EPI_NONE      : C bf16 = acc
 *            PW_EPI_BIAS      : C bf16 = acc + bias[n]
 *            PW_EPI_BIAS_RESID: C bf16 = acc + bias[n] + aux_in[m][n]          (aux_in bf16, ld_aux)
 *            PW_EPI_BIAS_GELU : C bf16 = acc + bias[n] (pre-activation) and aux_out bf16 = GeLU(that) (ldc)
 *            PW_EPI_DGELU     : C bf16 = acc * GeLU'(aux_in[m][n])             (aux_in bf16 = saved u)
 *            PW_EPI_F32       : C fp32 = acc, or C += acc when accumulate != 0
 * Leading dimensions are in elements; all of M, N, K multiples of 8; pointers 16-byte aligned. */
enum { PW_GEMM_TN = 0, PW_GEMM_NN = 1, PW_GEMM_NT = 2 };
enum { PW_EPI_NONE = 0, PW_EPI_BIAS = 1, PW_EPI_BIAS_RESID = 2, PW_EPI_BIAS_GELU = 3, PW_EPI_DGELU = 4,
       PW_EPI_F32 = 5 };
pw_status_t pw_op_gemm(int layout, int epilogue, int act, int M, int N, int K, const void* A, int lda,
                       const void* B, int ldb, void* C, int ldc, const void* bias, const void* aux_in,
                       int ld_aux, void* aux_out, int accumulate, void* stream);

/* Embedding lookup x0[t] = E[ids[t]] (bf16 rows of d elements, d % 8 == 0) and its backward
 * dE[ids[t]] += dx0[t] (fp32, tokens added in increasing t).  scratch: device,
 * pw_op_embedding_bwd_scratch_bytes(T, V) bytes. */
pw_status_t pw_op_embedding_fwd(const int32_t* ids, const void* E, int T, int d, int V, void* x0, void* stream);
size_t pw_op_embedding_bwd_scratch_bytes(int T, int V);
pw_status_t pw_op_embedding_bwd(const int32_t* ids, const void* dx0, int T, int d, int V, void* dE, void* scratch,
                                void* stream);
/* Softmax / cross-entropy over logits bf16 [T, ld] (V columns used, V % 8 == 0): lse fp32 [T],
 * loss_rows fp32 [T] = lse - logit[label]; the logits are replaced by
 * grad_scale * (softmax - onehot(label)). */
pw_status_t pw_op_softmax_xent(void* logits, int ld, const int32_t* labels, int T, int V, float grad_scale,
                               void* lse, void* loss_rows, void* stream);

/* The output projection's data gradient with the first step of attention backward folded into its
 * epilogue (the backward of Section 5.3's Transformer layer; the fusion itself is this library's):
 *   C bf16 [M,N] = A [M,K] B [K,N]   (PW_GEMM_NN operands: dout = dx1 Wo), and
 *   row_dot fp32 [M / seq_len, N / head_dim, seq_len]: row_dot[b][h][s] = sum over the head_dim
 *   columns c of head h of acc[b * seq_len + s][c] * other[b * seq_len + s][c], with acc the fp32
 *   product before it is rounded to bf16 and other bf16 [M,N] (row stride ld_other) = the attention
 *   output o; this is the rowsum(dO * O) that pw_op_attention_bwd otherwise computes itself.
 * head_dim 64 or 128 dividing N; seq_len dividing M; M, N, K multiples of 8; pointers 16-byte
 * aligned (row_dot: 4).  Errors: PW_ERR_CUDA with a message for a shape the GEMM refuses. */
pw_status_t pw_op_gemm_rowdot(int M, int N, int K, const void* A, int lda, const void* B, int ldb, void* C, int ldc,
                              const void* other, int ld_other, int head_dim, int seq_len, void* row_dot, void* stream);

/* Causal attention forward on packed qkv (bf16 [T,3d]); o bf16 [T,d]; lse fp32 [B,H,S].
 * The attention kernels are persistent and hand out their work through counters that live
 * beside the status word: the pw_op_attention_* calls of one device share one set, so two of them
 * must not run on the GPU at the same time (enqueue them on one stream, or order the streams). A
 * layer handle owns its own counters; different handles may overlap freely. */
pw_status_t pw_op_attention_fwd(const void* qkv, int B, int S, int H, int dh, void* o, void* lse, void* stream);

/* Causal attention backward.  dout bf16 [T,d]; dqkv bf16 [T,3d] (same packing as qkv);
 * delta: fp32 device scratch [B,H,S] (receives rowsum(dout*o)).  With o = NULL the call takes
 * delta as an input - already filled, e.g. by pw_op_gemm_rowdot - and launches two kernels
 * instead of three. */
pw_status_t pw_op_attention_bwd(const void* qkv, const void* o, const void* dout, const void* lse, int B, int S,
                                int H, int dh, void* dqkv, void* delta, void* stream);

/* Status word used by the pw_op_* calls (same meaning as pw_layer_status). */
pw_status_t pw_op_status(int* device_status, int* site);
/* y[i] = x[i] * scale + shift on fp32 device vectors (y may alias x).  The node type of the
 * paper's Figure 2 program (a(x) = x*2, b(x) = x+1, c(x) = x/2; f(v) = (b(a(v)), a(c(a(v))))): lets
 * that worked example run through the same enqueue-only / captured-graph dispatch as the layers. */
pw_status_t pw_op_affine_f32(const void* x, long long n, float scale, float shift, void* y, void* stream);
/* Gradient apply.  In the appendix's trace of data-parallel training each island applies the
 * gradients it received before the next step; the paper names no optimizer, so this is plain
 * stochastic gradient descent on an fp32 master copy with the bf16 working copy re-derived from it:
 *     master[i] <- master[i] - lr * grad_scale * grad[i]     (one fused multiply-add per element)
 *     param[i]   = bf16(master[i])                           (round to nearest even)
 * for every element of every item.  items is a HOST array of n_items entries; every pointer in it is
 * a DEVICE pointer owned by the caller: param bf16 [n] (read only when init_master != 0, always
 * written), master fp32 [n] (read unless init_master != 0, always written), grad fp32 [n] (read only;
 * e.g. a member of pw_layer_grads_t).  Items must not overlap.  init_master != 0 takes the old master
 * from param instead (first step, or lr = 0 to only create the master copy).  grad_scale is for
 * sums over micro-batches (1 / count).  Any alignment of the element type works; 16-byte aligned
 * tensors take the vector path.  Enqueue-only on `stream`; one launch per 64 items
 * (items with n == 0 do not count).
 * Errors: PW_ERR_INVALID_ARG for NULL / misaligned pointers, n < 0, n_items <= 0, lr < 0 or not
 * finite, grad_scale <= 0 or not finite; n == 0 items are skipped. */
typedef struct {
    void* param;       /* device, bf16 [n] */
    void* master;      /* device, fp32 [n] */
    const void* grad;  /* device, fp32 [n] */
    int64_t n;
} pw_apply_item_t;
pw_status_t pw_sgd_apply(const pw_apply_item_t* items, int n_items, float lr, float grad_scale, int init_master,
                         void* stream);
/* Data-parallel gradient apply over peer memory: the two-island data-parallel training of Section
 * 5.3 and the appendix trace (each island computes gradients, the islands exchange them, each
 * applies them), for replicas that are GPUs of one NVLink domain, one process each.  Every replica
 * keeps ALL its parameter gradients in one flat fp32 buffer and ALL its bf16 parameters in one flat
 * bf16 buffer (n_total elements each, same layout on every replica), both mapped into every other
 * replica (pw_shared_*).  Replica `rank` owns elements [lo, hi) (pw_dp_slice: equal slices, a
 * multiple of 8 elements) and holds the fp32 master of that slice only.  The call, for i in [lo, hi):
 *     g = grads[0][i] + grads[1][i] + ... + grads[world-1][i]      (fp32, this order)
 *     master_slice[i - lo] <- master_slice[i - lo] - lr * grad_scale * g
 *     params[k][i] = bf16(master_slice[i - lo])  for every replica k
 * i.e. reduce-scatter, step and all-gather of the working copy in one kernel of plain peer loads and
 * stores (no multicast, no waiting inside the kernel).  grads / params: HOST arrays of `world` DEVICE
 * pointers in rank order (entry `rank` is this replica's own buffer, the others are mapped peers).
 * init_master != 0 takes the old master from this replica's own params.
 * ORDERING IS THE CALLER'S: every replica's gradients must be complete before any replica's call
 * starts, and no replica may read params (next forward) or rewrite grads (next backward) before
 * every replica's call has finished - e.g. a one-element NCCL all-reduce on the same stream before
 * and after, or host barriers after a stream synchronize.  Enqueue-only on `stream`.
 * Errors: PW_ERR_INVALID_ARG for world outside [1, 8], a bad rank, NULL / misaligned buffers, bad
 * lr / grad_scale.  A replica whose slice is empty launches nothing. */
pw_status_t pw_dp_slice(int64_t n_total, int world, int rank, int64_t* lo, int64_t* hi);   /* host only, needs no GPU */
pw_status_t pw_dp_reduce_apply(int rank, int world, const void* const* grads, void* const* params, void* master_slice,
                               int64_t n_total, float lr, float grad_scale, int init_master, void* stream);
/* Device buffers that other processes can map (CUDA IPC).  pw_shared_alloc: cudaMalloc of `bytes` on
 * the current device plus a 64-byte handle to send to the other replicas (any host channel);
 * pw_shared_open: map another process's buffer (same GPU or a peer GPU of the node; peer access is
 * enabled on demand) - the handle's maker cannot open it itself; pw_shared_close / pw_shared_free
 * undo them.  Close every mapping before the owner frees the buffer. */
typedef struct { unsigned char bytes[64]; } pw_ipc_handle_t;
pw_status_t pw_shared_alloc(size_t bytes, void** dev_ptr, pw_ipc_handle_t* handle);
pw_status_t pw_shared_free(void* dev_ptr);
pw_status_t pw_shared_open(const pw_ipc_handle_t* handle, void** dev_ptr);
pw_status_t pw_shared_close(void* dev_ptr);
/* Process-wide tuning knobs.  The defaults are what the library is tested and measured with; a
 * measurement script flips one of them to take an A/B figure.  Not thread-safe; set them while no
 * call of this library is in progress.  A change invalidates the CUDA graphs that GRAPH dispatch
 * has cached (Section 5.1's Fused mode re-captures on its next call).  Values out of range and
 * unknown knobs return PW_ERR_INVALID_ARG and change nothing.
 *   PW_TUNE_PDL               1 (default) / 0: launch kernels with programmatic dependent launch
 *   PW_TUNE_GEMM_PAIR         1 (default) / 0: two-CTA 256 x 256 GEMM tiles whenever M >= 256
 *   PW_TUNE_GEMM_BN           0 (default: chosen per shape) / 128 / 192 / 256: forced GEMM tile width
 *   PW_TUNE_GEMM_SPLIT        1 (default) / 0: cut the tiles of a thin last round along K
 *   PW_TUNE_GEMM_SPLIT_MIN_K  64 (default): ... only from this many 64-wide K blocks on
 *   PW_TUNE_FAIL_LAUNCH       0 (default) / k > 0: host-side fault injection for error-path tests - the
 *                             k-th kernel launch from now is not enqueued and reports a launch failure
 *                             (the call that issued it returns PW_ERR_CUDA); the knob then returns to 0
 *   PW_TUNE_NVTX              0 (default) / 1: NVTX ranges ("pw_layer_fwd", "pw_layer_bwd",
 *                             "pw_stage_run_chain", "pw_lm_step", "pw_sgd_apply") around the host side of those
 *                             calls, for timeline tools; without a tool attached a range costs a function call */
enum {
    PW_TUNE_PDL = 0,
    PW_TUNE_GEMM_PAIR = 1,
    PW_TUNE_GEMM_BN = 2,
    PW_TUNE_GEMM_SPLIT = 3,
    PW_TUNE_GEMM_SPLIT_MIN_K = 4,
    PW_TUNE_FAIL_LAUNCH = 5,
    PW_TUNE_NVTX = 6
};
pw_status_t pw_set_tuning(int knob, int value);
pw_status_t pw_get_tuning(int knob, int* value);
/* Logging (the paper's monitoring side channel has no counterpart here; this is the library's own).
 * The library prints nothing by default.  pw_set_log installs a process-wide sink:
 *   level PW_LOG_OFF (default), PW_LOG_ERROR: every failure, with the text pw_last_error() would give;
 *   PW_LOG_INFO: also one line per pw_layer_create / pw_stage_create (shapes, workspace sizes) and per
 *   pw_stage_run_chain / pw_lm_step call (dispatch mode, layers, micro-batches).
 * fn(level, message, user) is called on the calling thread, before the failing call returns; message is
 * only valid during the call.  fn = NULL writes "pw: <message>" lines to stderr.  No environment
 * variable is read. */
enum { PW_LOG_OFF = 0, PW_LOG_ERROR = 1, PW_LOG_INFO = 2 };
typedef void (*pw_log_fn)(int level, const char* message, void* user);
pw_status_t pw_set_log(int level, pw_log_fn fn, void* user);

/* Clears the status word of the single-step calls (after a test has provoked an error). */
pw_status_t pw_op_status_reset(void);
/* Failure-path self-test.  Every device-side wait in this library is bounded; this call shows the
 * mechanism working without hanging anything: it launches one warp that waits on a barrier
 * nothing will ever signal, with a limit of limit_cycles SM cycles (clamped to [1e3, 2e9], i.e. at
 * most about a second).  The wait gives up, the status word of the single-step calls records
 * PW_ERR_TIMEOUT with site 990, and the kernel returns normally: *kernel_returned (host) = 1.
 * Synchronises the stream.  pw_op_status then reports (PW_ERR_TIMEOUT, 990) until
 * pw_op_status_reset. */
pw_status_t pw_op_selftest_wait_timeout(uint64_t limit_cycles, int* kernel_returned, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PW_H_ */
