// Internal launch interface between the host dispatch code and the kernels.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>

#include "pw_common.cuh"

namespace pw {

// Process-wide, per-device runtime state: SM count, the driver's tensor-map encoder, a default
// status block for the single-step entry points.
struct Runtime {
    int device = -1;
    int sm_count = 0;
    int cc_major = 0;
    void* encode_tiled = nullptr;      // cuTensorMapEncodeTiled, fetched through the runtime API
    void* split_ws = nullptr;          // split-K scratch of the single-step GEMM call (allocated with the runtime)
    DeviceStatus* op_status = nullptr; // device memory, status block for pw_op_* calls
};
// Returns nullptr (and sets *err) if the device is not sm_100 or a CUDA call failed.
Runtime* get_runtime(const char** err);

// One-time kernel attribute set-up (dynamic shared-memory opt-in); called from get_runtime.
const char* configure_gemm();
const char* configure_attention();
const char* configure_attention_fwd();
const char* configure_elementwise();

// Process-wide tuning knobs (pw_set_tuning); the defaults are what every measurement and test uses.
struct Tuning {
    int pdl = 1;                 // launch with the programmatic-serialization attribute
    int gemm_pair = 1;           // CTA-pair GEMM kernel whenever M >= 256
    int gemm_bn = 0;             // 0 = tile width chosen by the launcher, else 128 / 192 / 256
    int gemm_split = 1;          // cut the tiles of a thin last round along K
    int gemm_split_min_k = 64;   // ... from this many 64-wide K blocks on
    int nvtx = 0;                // NVTX ranges around the host side of the main entry points
    uint64_t epoch = 0;          // bumped by every change (part of the CUDA-graph cache key)
    // Host-side fault injection for the error-path tests: when > 0, counts down once per launch and
    // the launch that brings it to zero is NOT enqueued and reports cudaErrorLaunchFailure instead.
    int fail_launch_countdown = 0;
};
Tuning& tuning();

// Launch with the programmatic-serialization attribute (see grid_dep_wait in pw_common.cuh).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args)
{
    Tuning& tn = tuning();
    if (tn.fail_launch_countdown > 0 && --tn.fail_launch_countdown == 0) return cudaErrorLaunchFailure;   // injected by a test
    const bool pdl = tn.pdl != 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

enum GemmLayout { kTN = 0, kNN = 1, kNT = 2 };
enum GemmEpi { kEpiNone = 0, kEpiBias = 1, kEpiBiasResid = 2, kEpiBiasGelu = 3, kEpiDGelu = 4, kEpiF32 = 5,
               kEpiRowDot = 6 /* C bf16 = acc, and rowdot[b][h][s] = sum over the columns of head h of acc * aux_in */ };

struct GemmArgs {
    int layout, epilogue, act;
    int M, N, K;
    const void* A; int lda;
    const void* B; int ldb;
    void* C; int ldc;
    const void* bias;
    const void* aux_in; int ld_aux;
    void* aux_out;
    int accumulate;
    // Optional fp32 scratch of gemm_split_ws_bytes(): lets the tiles of a thin last round be cut in two
    // along K.  Only for GEMMs that never run beside another GEMM using the same status word.
    void* split_ws = nullptr;
    // kEpiRowDot (the output projection's data gradient, C = dO): per (row, head) dot products of the
    // fp32 result with aux_in (= O) go to row_dot as fp32 [B, H, S], rows being tokens b * S + s and
    // heads head_dim consecutive columns - the rowsum(dO * O) that attention backward starts from.
    void* row_dot = nullptr; int head_dim = 0, seq_len = 0;
};
size_t gemm_split_ws_bytes();
// Encodes the two tensor maps and launches.  Returns nullptr on success, else a static message.
const char* launch_gemm(Runtime* rt, const GemmArgs& a, DeviceStatus* status, cudaStream_t stream);

const char* launch_layernorm_fwd(Runtime* rt, const void* x, const void* gamma, const void* beta, int T, int d,
                                 float eps, void* h, void* mu, void* rstd, cudaStream_t stream);
size_t layernorm_bwd_scratch_bytes(Runtime* rt, int T, int d);
const char* launch_layernorm_bwd(Runtime* rt, const void* dh, const void* x, const void* mu, const void* rstd,
                                 const void* gamma, const void* resid, int T, int d, void* dx, void* dgamma,
                                 void* dbeta, void* db_resid, void* db_dx, int accumulate, void* partials,
                                 cudaStream_t stream);
size_t colsum_scratch_bytes(Runtime* rt, int T, int N);
const char* launch_colsum(Runtime* rt, const void* in, int T, int N, int ld, void* out, int accumulate,
                          void* partials, cudaStream_t stream);

// The LayerNorm backward and the column-sum kernels leave one partial row per CTA slot; a second,
// fixed-order kernel adds them up.  The *_partial launchers run the first kernel only and describe
// the second in a ReduceJob, so that a caller with several of them (a layer's backward has four)
// can finish them all with one launch_reduce_jobs - at most kReduceMaxEntries output vectors.
constexpr int kReduceMaxEntries = 8;
struct ReduceJob {
    const float* partials;      // [nrows][nq][n]
    int nrows, nq, n;
    float* out[4];              // out[q] (+)= sum over rows of partials[.][q][.]; nullptr: skip
};
const char* launch_layernorm_bwd_partial(Runtime* rt, const void* dh, const void* x, const void* mu, const void* rstd,
                                         const void* gamma, const void* resid, int T, int d, void* dx, void* dgamma,
                                         void* dbeta, void* db_resid, void* db_dx, void* partials, ReduceJob* job,
                                         cudaStream_t stream);
const char* launch_colsum_partial(Runtime* rt, const void* in, int T, int N, int ld, void* out, void* partials,
                                  ReduceJob* job, cudaStream_t stream);
const char* launch_reduce_jobs(const ReduceJob* jobs, int njobs, int accumulate, cudaStream_t stream);

// Column sums with the partial sums in a fixed device array inside the library (no allocation, no Runtime).
size_t colsum_noalloc_max_columns();
// On failure *err_kind says what went wrong: an argument, the device (not sm_100) or a CUDA call.
enum { kErrArgument = 0, kErrDevice = 1, kErrCuda = 2 };
const char* launch_colsum_noalloc(const void* in, int T, int N, int ld, void* out, int accumulate, cudaStream_t stream,
                                  int* err_kind);

// a = GeLU(u), bf16 -> bf16, n a multiple of 8.
const char* launch_gelu_fwd(Runtime* rt, const void* u, void* a, long long n, int act, cudaStream_t stream);

const char* launch_affine_f32(const void* x, long long n, float scale, float shift, void* y, cudaStream_t stream);

// Gradient apply (optimizer.cu): master -= step * grad, param = bf16(master), for every item; with
// init_master the old master is taken from param instead of being read.
constexpr int kApplyMaxItems = 64;                      // tensors served by one launch
struct ApplyItem { void* param; void* master; const void* grad; long long n; };
const char* launch_sgd_apply(const ApplyItem* items, int n_items, float step, int init_master, cudaStream_t stream);

// Data-parallel gradient apply over peer memory (optimizer.cu).  grads / params: host arrays of `world`
// device pointers (flat fp32 gradient and bf16 parameter buffers of every replica, n_total elements
// each); master: this replica's fp32 slice [lo, hi) as given by dp_slice.
constexpr int kDpMaxWorld = 8;
void dp_slice(long long n_total, int world, int rank, long long* lo, long long* hi);
const char* launch_dp_reduce_apply(int rank, int world, const void* const* grads, void* const* params, void* master,
                                   long long n_total, float step, int init_master, cudaStream_t stream);

// Bounded-wait self-test (selftest.cu): *returned (device int) becomes 1 when the wait gave up and the kernel went on.
const char* launch_wait_selftest(DeviceStatus* status, long long limit, int* returned, cudaStream_t stream);

// First / last layer of the language model (lm_head.cu).
const char* launch_embedding_fwd(Runtime* rt, const void* ids, const void* E, int T, int d, int V, void* x0,
                                 DeviceStatus* status, cudaStream_t stream);
size_t embedding_bwd_scratch_bytes(int T, int V);
const char* launch_embedding_bwd(Runtime* rt, const void* ids, const void* dx0, int T, int d, int V, void* dE,
                                 void* scratch, DeviceStatus* status, cudaStream_t stream);
const char* launch_softmax_xent(Runtime* rt, void* logits, int ld, const void* labels, int T, int V, float grad_scale,
                                void* lse, void* loss_rows, DeviceStatus* status, cudaStream_t stream);
const char* launch_sum_scale(const void* in, int n, float scale, void* out, cudaStream_t stream);

const char* launch_attention_fwd(Runtime* rt, const void* qkv, int B, int S, int H, int dh, void* o, void* lse,
                                 DeviceStatus* status, cudaStream_t stream);
const char* launch_attention_bwd(Runtime* rt, const void* qkv, const void* o, const void* dout, const void* lse,
                                 int B, int S, int H, int dh, void* dqkv, void* delta, DeviceStatus* status,
                                 cudaStream_t stream);

// The layer's forward or backward as one cooperative launch (whole_layer.cu), for small shapes.
// Tensor names are those of the layer plan: ctx tensors (h1 ... r2), backward temporaries (big =
// du, later dqkv; td0 = dh2, dout, dh1; dx1), the 12 parameters and their fp32 gradients.
constexpr int kWholeLayerMaxTiles = 1024;           // (tokens / 64) * (d_model / 64): one split-K ticket each
struct WholeLayerArgs {
    int T, d, H, F, B, S, act, accumulate, with_fc2;
    int split_o, split_fc2, split_dh2, split_dh1;   // K slices of the GEMMs with [T, d] outputs (set by the launcher)
    float eps, scale;
    const void *x, *dy;
    void *y, *dx;
    const void *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_o, *b_o, *ln2_g, *ln2_b, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
    void *h1, *qkv, *o, *x1, *h2, *u, *a, *lse, *mu1, *r1, *mu2, *r2;
    void *big, *td0, *dx1;
    void *g_ln1_g, *g_ln1_b, *g_w_qkv, *g_b_qkv, *g_w_o, *g_b_o, *g_ln2_g, *g_ln2_b, *g_w_fc1, *g_b_fc1, *g_w_fc2, *g_b_fc2;
    void* splitk;                                   // whole_layer_splitk_bytes() of fp32 partial tiles
    unsigned* sync;                                 // 2 + kWholeLayerMaxTiles words, zero when the handle is created
    DeviceStatus* status;
};
const char* configure_whole_layer();
const char* whole_layer_unsupported(int T, int d, int H, int dh, int F, int S);   // nullptr if the shape is served
size_t whole_layer_splitk_bytes(int T, int d);
const char* launch_whole_layer(Runtime* rt, WholeLayerArgs a, bool backward, cudaStream_t stream);

}  // namespace pw
