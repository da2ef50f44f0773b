// C ABI of the decoder-layer engine: runtime set-up, static launch plans, asynchronous enqueue
// of one layer's forward / backward, and the stage chain with its three dispatch modes.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <cstddef>
#include <cmath>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/pw.h"
#include "pw_kernels.h"

namespace pw {

static thread_local std::string g_last_error;

Tuning& tuning()
{
    static Tuning t;
    return t;
}

// Log sink (pw_set_log): process-wide, guarded by a mutex; nothing is printed unless a level is set.
struct LogSink { int level = 0; pw_log_fn fn = nullptr; void* user = nullptr; };
static LogSink g_log;
static std::mutex g_log_mu;
static void log_line(int level, const std::string& msg)
{
    LogSink sink;
    {
        std::lock_guard<std::mutex> lock(g_log_mu);
        sink = g_log;
    }
    if (sink.level < level) return;
    if (sink.fn) sink.fn(level, msg.c_str(), sink.user);
    else fprintf(stderr, "pw: %s\n", msg.c_str());
}
static bool log_enabled(int level)
{
    std::lock_guard<std::mutex> lock(g_log_mu);
    return g_log.level >= level;
}

static pw_status_t fail(pw_status_t s, const std::string& msg)
{
    g_last_error = msg;
    log_line(PW_LOG_ERROR, std::string(pw_status_string(s)) + ": " + msg);
    return s;
}

// NVTX range around the host side of an entry point (PW_TUNE_NVTX); the v3 header needs no library.
struct NvtxRange {
    bool on;
    explicit NvtxRange(const char* name) : on(tuning().nvtx != 0) { if (on) nvtxRangePushA(name); }
    ~NvtxRange() { if (on) nvtxRangePop(); }
};
static pw_status_t fail_cuda(const char* what, cudaError_t e)
{
    return fail(PW_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

Runtime* get_runtime(const char** err)
{
    static std::mutex mu;
    static std::map<int, Runtime*> per_device;
    std::lock_guard<std::mutex> lock(mu);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { *err = "no CUDA device (cudaGetDevice failed)"; return nullptr; }
    auto it = per_device.find(dev);
    if (it != per_device.end()) return it->second;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { *err = "cudaGetDeviceProperties failed"; return nullptr; }
    if (prop.major != 10) { *err = "device is not compute capability 10.x (sm_100a kernels only, no fallback)"; return nullptr; }
    Runtime* rt = new Runtime();
    rt->device = dev;
    rt->sm_count = prop.multiProcessorCount;
    rt->cc_major = prop.major;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &rt->encode_tiled, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || rt->encode_tiled == nullptr) {
        delete rt; *err = "cuTensorMapEncodeTiled not available from the driver"; return nullptr;
    }
    const char* ce;
    if ((ce = configure_gemm()) || (ce = configure_attention()) || (ce = configure_attention_fwd()) || (ce = configure_elementwise()) || (ce = configure_whole_layer())) { delete rt; *err = ce; return nullptr; }
    if (cudaMalloc(reinterpret_cast<void**>(&rt->op_status), sizeof(DeviceStatus)) != cudaSuccess ||
        cudaMemset(rt->op_status, 0, sizeof(DeviceStatus)) != cudaSuccess) {
        delete rt; *err = "could not allocate the status word"; return nullptr;
    }
    // split-K scratch of the single-step GEMM call; without it that call simply never cuts a tile
    if (cudaMalloc(&rt->split_ws, gemm_split_ws_bytes()) != cudaSuccess) { rt->split_ws = nullptr; (void)cudaGetLastError(); }
    per_device[dev] = rt;
    return rt;
}

static inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

// Static plan of one layer: shapes, workspace offsets.
struct LayerPlan {
    pw_layer_config_t cfg;
    int T, d, H, dh, F, B, S;
    float eps;
    size_t ctx_off[PW_CTX_COUNT], ctx_size[PW_CTX_COUNT], ctx_bytes;
    // scratch = [ctx-shaped region used when the caller passes ctx == NULL] [backward temporaries]
    size_t off_big, off_td0, off_td1, off_delta, off_partials, off_partials2, off_partials3, off_partials4, scratch_bytes;
    // lean ctx: h1, h2, a (and the statistics the re-derivation writes again) live in scratch
    bool lean;
    size_t off_lean_h1, off_lean_h2, off_lean_a, off_lean_stats;
    size_t off_splitk;           // partial sums of GEMM tiles cut along K (main-stream GEMMs only)
    // PW_FLAG_WHOLE_LAYER: forward and backward are one cooperative launch each
    bool whole;
    size_t off_whole_splitk;
};

}  // namespace pw

struct pw_layer {
    pw::LayerPlan plan;
    pw::Runtime* rt;
    pw::DeviceStatus* status;
    unsigned* whole_sync = nullptr; // grid-barrier and split-K words of the whole-layer kernels (zero between launches)
    cudaStream_t aux = nullptr;     // side stream: weight gradients and bias column sums run beside the dgrad chain
    cudaEvent_t ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    uint64_t launches = 0;          // kernels launched (or replayed) through this handle
    bool single_stream = false;     // pw_layer_set_side_stream(layer, 0): everything on the calling stream
    bool capturing = false;         // inside a stream capture: count launches into graph_nodes instead
    uint64_t graph_nodes = 0;
    // profiling: event pairs around every launch group
    bool profiling = false;
    struct Span { cudaEvent_t a, b; int cls; };
    std::vector<Span> spans;
    std::vector<cudaEvent_t> pool;
    cudaStream_t prof_stream = nullptr;
    pw_profile_t prof;
};

struct pw_stage {
    pw_layer_t* layer;
    int n_layers;
    struct Cached { cudaGraphExec_t exec; uint64_t nodes; };
    std::map<std::vector<uint64_t>, Cached> graphs;
};

namespace pw {

static pw_status_t validate_cfg(const pw_layer_config_t* c)
{
    if (!c) return fail(PW_ERR_INVALID_ARG, "config is NULL");
    if (c->struct_size != sizeof(pw_layer_config_t)) return fail(PW_ERR_INVALID_ARG, "config struct_size mismatch");
    if (c->d_model <= 0 || c->n_heads <= 0 || c->head_dim <= 0 || c->d_ff <= 0 || c->seq_len <= 0 || c->batch <= 0)
        return fail(PW_ERR_INVALID_ARG, "config has a non-positive dimension");
    if (c->act != PW_ACT_GELU_ERF && c->act != PW_ACT_GELU_TANH) return fail(PW_ERR_INVALID_ARG, "unknown activation");
    if (c->causal != 1) return fail(PW_ERR_UNSUPPORTED_SHAPE, "only causal attention is supported");
    if ((c->flags & ~static_cast<uint32_t>(PW_FLAG_LEAN_CTX | PW_FLAG_WHOLE_LAYER)) != 0) return fail(PW_ERR_INVALID_ARG, "unknown flag");
    if ((c->flags & PW_FLAG_LEAN_CTX) && (c->flags & PW_FLAG_WHOLE_LAYER))
        return fail(PW_ERR_INVALID_ARG, "PW_FLAG_LEAN_CTX and PW_FLAG_WHOLE_LAYER exclude one another");
    if (c->ln_eps < 0.f) return fail(PW_ERR_INVALID_ARG, "ln_eps must be >= 0");
    if (c->head_dim != 64 && c->head_dim != 128) return fail(PW_ERR_UNSUPPORTED_SHAPE, "head_dim must be 64 or 128");
    if (static_cast<long long>(c->n_heads) * c->head_dim != c->d_model)
        return fail(PW_ERR_UNSUPPORTED_SHAPE, "n_heads * head_dim must equal d_model");
    if (c->d_model % 256 != 0 || c->d_model > 8192) return fail(PW_ERR_UNSUPPORTED_SHAPE, "d_model must be a multiple of 256, at most 8192");
    if (c->d_ff % 128 != 0) return fail(PW_ERR_UNSUPPORTED_SHAPE, "d_ff must be a multiple of 128");
    if (c->seq_len % 128 != 0) return fail(PW_ERR_UNSUPPORTED_SHAPE, "seq_len must be a multiple of 128");
    if (static_cast<long long>(c->batch) * c->seq_len > (1ll << 24)) return fail(PW_ERR_UNSUPPORTED_SHAPE, "too many tokens per call");
    if (c->flags & PW_FLAG_WHOLE_LAYER) {
        const char* why = whole_layer_unsupported(c->batch * c->seq_len, c->d_model, c->n_heads, c->head_dim, c->d_ff, c->seq_len);
        if (why) return fail(PW_ERR_UNSUPPORTED_SHAPE, why);
    }
    return PW_OK;
}

static void build_plan(const pw_layer_config_t& c, Runtime* rt, LayerPlan* p)
{
    p->cfg = c;
    p->B = c.batch; p->S = c.seq_len; p->T = c.batch * c.seq_len;
    p->d = c.d_model; p->H = c.n_heads; p->dh = c.head_dim; p->F = c.d_ff;
    p->eps = c.ln_eps > 0.f ? c.ln_eps : 1e-5f;
    const size_t T = p->T, d = p->d, F = p->F;
    p->lean = (c.flags & PW_FLAG_LEAN_CTX) != 0;
    size_t sz[PW_CTX_COUNT] = {T * d * 2, T * 3 * d * 2, T * d * 2, T * d * 2, T * d * 2, T * F * 2, T * F * 2,
                               static_cast<size_t>(p->B) * p->H * p->S * 4, T * 4, T * 4, T * 4, T * 4};
    if (p->lean) sz[PW_CTX_H1] = sz[PW_CTX_H2] = sz[PW_CTX_A] = 0;
    size_t off = 0;
    for (int i = 0; i < PW_CTX_COUNT; ++i) { p->ctx_off[i] = off; p->ctx_size[i] = sz[i]; off += align256(sz[i]); }
    p->ctx_bytes = off;
    size_t s = p->ctx_bytes;
    p->off_big = s; s += align256((F > 3 * d ? T * F : T * 3 * d) * 2);
    p->off_td0 = s; s += align256(T * d * 2);
    p->off_td1 = s; s += align256(T * d * 2);
    p->off_delta = s; s += align256(static_cast<size_t>(p->B) * p->H * p->S * 4);
    size_t part = layernorm_bwd_scratch_bytes(rt, p->T, p->d);
    const size_t c1 = colsum_scratch_bytes(rt, p->T, p->F), c2 = colsum_scratch_bytes(rt, p->T, 3 * p->d);
    if (c1 > part) part = c1;
    if (c2 > part) part = c2;
    p->off_partials = s; s += align256(part);
    // The four sets of partial rows of a backward call (LN2, LN1, the two bias column sums) are
    // summed by one launch at the end of the call, so each has a region of its own.
    p->off_partials2 = s; s += align256(c1);                                           // db1 column sums (side stream)
    p->off_partials3 = s; s += align256(layernorm_bwd_scratch_bytes(rt, p->T, p->d));  // LN1 backward
    p->off_partials4 = s; s += align256(c2);                                           // dbqkv column sums (side stream)
    p->off_splitk = s; s += align256(gemm_split_ws_bytes());
    p->off_lean_h1 = p->off_lean_h2 = p->off_lean_a = p->off_lean_stats = 0;
    if (p->lean) {
        p->off_lean_h1 = s; s += align256(T * d * 2);
        p->off_lean_h2 = s; s += align256(T * d * 2);
        p->off_lean_a = s; s += align256(T * F * 2);
        p->off_lean_stats = s; s += 2 * align256(T * 4);
    }
    p->whole = (c.flags & PW_FLAG_WHOLE_LAYER) != 0;
    p->off_whole_splitk = 0;
    if (p->whole) { p->off_whole_splitk = s; s += align256(whole_layer_splitk_bytes(p->T, p->d)); }
    p->scratch_bytes = s;
}

// Runs one launch group, counting its kernels and (when profiling) bracketing it with events.
struct LaunchScope {
    pw_layer_t* L; int cls; cudaStream_t st; cudaEvent_t a = nullptr, b = nullptr;
    static cudaEvent_t get_event(pw_layer_t* L)
    {
        if (!L->pool.empty()) { cudaEvent_t e = L->pool.back(); L->pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
    LaunchScope(pw_layer_t* L_, int cls_, int nkernels, double flops, double bytes, cudaStream_t st_)
        : L(L_), cls(cls_), st(st_)
    {
        if (L->capturing) L->graph_nodes += nkernels; else L->launches += nkernels;
        if (L->profiling) {
            L->prof.launches[cls] += nkernels; L->prof.flops[cls] += flops; L->prof.bytes[cls] += bytes;
            L->prof_stream = st;
            a = get_event(L); b = get_event(L);
            if (a) cudaEventRecord(a, st);
        }
    }
    ~LaunchScope()
    {
        if (L->profiling && a && b) { cudaEventRecord(b, st); L->spans.push_back({a, b, cls}); }
    }
    // The launch group failed before anything was enqueued: take its kernels out of the counts again.
    void cancel(int nkernels)
    {
        if (L->capturing) L->graph_nodes -= nkernels; else L->launches -= nkernels;
        if (L->profiling) L->prof.launches[cls] -= nkernels;
    }
};

static inline uint8_t* at(void* base, size_t off) { return static_cast<uint8_t*>(base) + off; }
static inline const uint8_t* at(const void* base, size_t off) { return static_cast<const uint8_t*>(base) + off; }

static GemmArgs gemm_args(int layout, int epi, int act, int M, int N, int K, const void* A, int lda, const void* B,
                          int ldb, void* C, int ldc, const void* bias, const void* aux_in, int ld_aux, void* aux_out,
                          int accumulate, void* split_ws = nullptr)
{
    GemmArgs g;
    g.split_ws = split_ws;
    g.layout = layout; g.epilogue = epi; g.act = act; g.M = M; g.N = N; g.K = K;
    g.A = A; g.lda = lda; g.B = B; g.ldb = ldb; g.C = C; g.ldc = ldc;
    g.bias = bias; g.aux_in = aux_in; g.ld_aux = ld_aux; g.aux_out = aux_out; g.accumulate = accumulate;
    return g;
}

#define PW_DO(expr)                          \
    do {                                     \
        pw_status_t s__ = (expr);            \
        if (s__ != PW_OK) return s__;        \
    } while (0)

static pw_status_t do_gemm(pw_layer_t* L, const GemmArgs& g, cudaStream_t st)
{
    const int cls = g.layout == kTN ? PW_K_GEMM_TN : g.layout == kNN ? PW_K_GEMM_NN : PW_K_GEMM_NT;
    LaunchScope sc(L, cls, 1, 2.0 * g.M * g.N * g.K, 0.0, st);
    const char* e = launch_gemm(L->rt, g, L->status, st);
    if (e) sc.cancel(1);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}
static pw_status_t do_ln_fwd(pw_layer_t* L, const void* x, const void* gamma, const void* beta, void* h, void* mu,
                             void* rstd, cudaStream_t st)
{
    const LayerPlan& p = L->plan;
    LaunchScope sc(L, PW_K_LN_FWD, 1, 0.0, 4.0 * p.T * p.d + 8.0 * p.T, st);
    const char* e = launch_layernorm_fwd(L->rt, x, gamma, beta, p.T, p.d, p.eps, h, mu, rstd, st);
    if (e) sc.cancel(1);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}
static pw_status_t do_ln_bwd(pw_layer_t* L, const void* dh, const void* x, const void* mu, const void* rstd,
                             const void* gamma, const void* resid, void* dx, void* dgamma, void* dbeta, void* db_resid,
                             void* db_dx, int accumulate, void* partials, cudaStream_t st, ReduceJob* defer = nullptr)
{
    // defer: the partial rows are left for a later launch_reduce_jobs (the caller collects the jobs)
    const LayerPlan& p = L->plan;
    LaunchScope sc(L, PW_K_LN_BWD, defer ? 1 : 2, 0.0, 8.0 * p.T * p.d + 8.0 * p.T, st);
    const char* e = defer
        ? launch_layernorm_bwd_partial(L->rt, dh, x, mu, rstd, gamma, resid, p.T, p.d, dx, dgamma, dbeta, db_resid, db_dx,
                                       partials, defer, st)
        : launch_layernorm_bwd(L->rt, dh, x, mu, rstd, gamma, resid, p.T, p.d, dx, dgamma, dbeta, db_resid, db_dx,
                               accumulate, partials, st);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}
static pw_status_t do_colsum(pw_layer_t* L, const void* in, int N, void* out, int accumulate, void* partials,
                             cudaStream_t st, ReduceJob* defer = nullptr)
{
    const LayerPlan& p = L->plan;
    LaunchScope sc(L, PW_K_COLSUM, defer ? 1 : 2, 0.0, 2.0 * p.T * N, st);
    const char* e = defer ? launch_colsum_partial(L->rt, in, p.T, N, N, out, partials, defer, st)
                          : launch_colsum(L->rt, in, p.T, N, N, out, accumulate, partials, st);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}
static pw_status_t do_reduce(pw_layer_t* L, const ReduceJob* jobs, int njobs, int accumulate, cudaStream_t st)
{
    double bytes = 0.0;                                  // the partial rows it reads (they are still in L2 more often than not)
    for (int j = 0; j < njobs; ++j) bytes += 4.0 * jobs[j].nrows * jobs[j].nq * jobs[j].n;
    LaunchScope sc(L, PW_K_REDUCE, 1, 0.0, bytes, st);
    const char* e = launch_reduce_jobs(jobs, njobs, accumulate, st);
    if (e) sc.cancel(1);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}
// Attention FLOPs count the visible (causal) pairs only: 2 T (S+1) d forward, 2.5x that backward.
static pw_status_t do_attn_fwd(pw_layer_t* L, const void* qkv, void* o, void* lse, cudaStream_t st)
{
    const LayerPlan& p = L->plan;
    LaunchScope sc(L, PW_K_ATTN_FWD, 1, 2.0 * p.T * (p.S + 1.0) * p.d, 0.0, st);
    const char* e = launch_attention_fwd(L->rt, qkv, p.B, p.S, p.H, p.dh, o, lse, L->status, st);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}
static pw_status_t do_attn_bwd(pw_layer_t* L, const void* qkv, const void* o, const void* dout, const void* lse,
                               void* dqkv, void* delta, cudaStream_t st)
{
    const LayerPlan& p = L->plan;
    const int nk = o ? 3 : 2;                            // o == nullptr: delta was filled by the GEMM that made dout
    LaunchScope sc(L, PW_K_ATTN_BWD, nk, 5.0 * p.T * (p.S + 1.0) * p.d, 0.0, st);
    const char* e = launch_attention_bwd(L->rt, qkv, o, dout, lse, p.B, p.S, p.H, p.dh, dqkv, delta, L->status, st);
    if (e) sc.cancel(nk);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}

// One launch for the whole forward (or backward) of a PW_FLAG_WHOLE_LAYER handle.
static pw_status_t do_whole_layer(pw_layer_t* L, const pw_layer_params_t* P, const void* x, void* y, const void* dy, void* dx,
                                  const pw_layer_grads_t* G, int accumulate, void* ctx, void* scratch, bool with_fc2,
                                  bool backward, cudaStream_t st)
{
    const LayerPlan& p = L->plan;
    WholeLayerArgs a = {};
    a.T = p.T; a.d = p.d; a.H = p.H; a.F = p.F; a.B = p.B; a.S = p.S; a.act = p.cfg.act;
    a.accumulate = accumulate; a.with_fc2 = with_fc2 ? 1 : 0;
    a.eps = p.eps; a.scale = 1.0f / sqrtf(static_cast<float>(p.dh));
    a.x = x; a.y = y; a.dy = dy; a.dx = dx;
    a.ln1_g = P->ln1_gamma; a.ln1_b = P->ln1_beta; a.w_qkv = P->w_qkv; a.b_qkv = P->b_qkv; a.w_o = P->w_o; a.b_o = P->b_o;
    a.ln2_g = P->ln2_gamma; a.ln2_b = P->ln2_beta; a.w_fc1 = P->w_fc1; a.b_fc1 = P->b_fc1; a.w_fc2 = P->w_fc2; a.b_fc2 = P->b_fc2;
    a.h1 = at(ctx, p.ctx_off[PW_CTX_H1]); a.qkv = at(ctx, p.ctx_off[PW_CTX_QKV]); a.o = at(ctx, p.ctx_off[PW_CTX_O]);
    a.x1 = at(ctx, p.ctx_off[PW_CTX_X1]); a.h2 = at(ctx, p.ctx_off[PW_CTX_H2]); a.u = at(ctx, p.ctx_off[PW_CTX_U]);
    a.a = at(ctx, p.ctx_off[PW_CTX_A]); a.lse = at(ctx, p.ctx_off[PW_CTX_LSE]);
    a.mu1 = at(ctx, p.ctx_off[PW_CTX_MU1]); a.r1 = at(ctx, p.ctx_off[PW_CTX_R1]);
    a.mu2 = at(ctx, p.ctx_off[PW_CTX_MU2]); a.r2 = at(ctx, p.ctx_off[PW_CTX_R2]);
    a.big = at(scratch, p.off_big); a.td0 = at(scratch, p.off_td0); a.dx1 = at(scratch, p.off_td1);
    if (G) {
        a.g_ln1_g = G->ln1_gamma; a.g_ln1_b = G->ln1_beta; a.g_w_qkv = G->w_qkv; a.g_b_qkv = G->b_qkv; a.g_w_o = G->w_o;
        a.g_b_o = G->b_o; a.g_ln2_g = G->ln2_gamma; a.g_ln2_b = G->ln2_beta; a.g_w_fc1 = G->w_fc1; a.g_b_fc1 = G->b_fc1;
        a.g_w_fc2 = G->w_fc2; a.g_b_fc2 = G->b_fc2;
    }
    a.splitk = at(scratch, p.off_whole_splitk);
    a.sync = L->whole_sync;
    a.status = L->status;
    const double T = p.T, d = p.d, F = p.F;
    const double fwd_flops = 2.0 * T * d * (4.0 * d + 2.0 * F) + 2.0 * T * (p.S + 1.0) * d;
    LaunchScope sc(L, PW_K_WHOLE_LAYER, 1, backward ? 2.0 * fwd_flops + T * (p.S + 1.0) * d : fwd_flops, 0.0, st);
    const char* e = launch_whole_layer(L->rt, a, backward, st);
    if (e) sc.cancel(1);
    return e ? fail(PW_ERR_CUDA, e) : PW_OK;
}

// Forward into `ctx` (a ctx-shaped region).  with_fc2 = false stops after FC1/GeLU (all that a
// recomputing backward needs).
static pw_status_t enqueue_fwd(pw_layer_t* L, const pw_layer_params_t* P, const void* x, void* y, void* ctx,
                               void* scratch, bool with_fc2, cudaStream_t st)
{
    const LayerPlan& p = L->plan;
    if (p.whole) return do_whole_layer(L, P, x, y, nullptr, nullptr, nullptr, 0, ctx, scratch, with_fc2, false, st);
    const int T = p.T, d = p.d, F = p.F, act = p.cfg.act;
    void* h1 = p.lean ? at(scratch, p.off_lean_h1) : at(ctx, p.ctx_off[PW_CTX_H1]);
    void* h2 = p.lean ? at(scratch, p.off_lean_h2) : at(ctx, p.ctx_off[PW_CTX_H2]);
    void* a = p.lean ? at(scratch, p.off_lean_a) : at(ctx, p.ctx_off[PW_CTX_A]);
    void* qkv = at(ctx, p.ctx_off[PW_CTX_QKV]);
    void* o = at(ctx, p.ctx_off[PW_CTX_O]);     void* x1 = at(ctx, p.ctx_off[PW_CTX_X1]);
    void* u = at(ctx, p.ctx_off[PW_CTX_U]);     void* lse = at(ctx, p.ctx_off[PW_CTX_LSE]);
    void* mu1 = at(ctx, p.ctx_off[PW_CTX_MU1]); void* r1 = at(ctx, p.ctx_off[PW_CTX_R1]);
    void* mu2 = at(ctx, p.ctx_off[PW_CTX_MU2]); void* r2 = at(ctx, p.ctx_off[PW_CTX_R2]);

    // GEMMs on the calling stream never overlap one another, so they may use the split-K scratch.
    void* sk = scratch ? at(scratch, p.off_splitk) : nullptr;
    PW_DO(do_ln_fwd(L, x, P->ln1_gamma, P->ln1_beta, h1, mu1, r1, st));
    PW_DO(do_gemm(L, gemm_args(kTN, kEpiBias, act, T, 3 * d, d, h1, d, P->w_qkv, d, qkv, 3 * d, P->b_qkv,
                                     nullptr, 0, nullptr, 0, sk), st));
    PW_DO(do_attn_fwd(L, qkv, o, lse, st));
    PW_DO(do_gemm(L, gemm_args(kTN, kEpiBiasResid, act, T, d, d, o, d, P->w_o, d, x1, d, P->b_o, x, d,
                                     nullptr, 0, sk), st));
    PW_DO(do_ln_fwd(L, x1, P->ln2_gamma, P->ln2_beta, h2, mu2, r2, st));
    PW_DO(do_gemm(L, gemm_args(kTN, kEpiBiasGelu, act, T, F, d, h2, d, P->w_fc1, d, u, F, P->b_fc1, nullptr, 0,
                                     a, 0, sk), st));
    if (with_fc2)
        PW_DO(do_gemm(L, gemm_args(kTN, kEpiBiasResid, act, T, d, F, a, F, P->w_fc2, F, y, d, P->b_fc2, x1, d,
                                         nullptr, 0, sk), st));
    return PW_OK;
}

static pw_status_t enqueue_bwd(pw_layer_t* L, const pw_layer_params_t* P, const void* x, const void* dy, void* dx,
                               const pw_layer_grads_t* G, int accumulate, const void* ctx, void* scratch,
                               cudaStream_t st)
{
    const LayerPlan& p = L->plan;
    const int T = p.T, d = p.d, F = p.F, act = p.cfg.act;
    bool rederive = p.lean;                              // h1, h2, a are not in a lean ctx
    if (ctx == nullptr) {
        pw_status_t s = enqueue_fwd(L, P, x, nullptr, scratch, scratch, false, st);
        if (s != PW_OK) return s;
        ctx = scratch;
        rederive = false;                                // the forward that just ran left them in scratch
    }
    if (p.whole) return do_whole_layer(L, P, x, nullptr, dy, dx, G, accumulate, const_cast<void*>(ctx), scratch, false, true, st);
    const void* h1 = p.lean ? at(scratch, p.off_lean_h1) : at(ctx, p.ctx_off[PW_CTX_H1]);
    const void* h2 = p.lean ? at(scratch, p.off_lean_h2) : at(ctx, p.ctx_off[PW_CTX_H2]);
    const void* a = p.lean ? at(scratch, p.off_lean_a) : at(ctx, p.ctx_off[PW_CTX_A]);
    const void* qkv = at(ctx, p.ctx_off[PW_CTX_QKV]);
    const void* o = at(ctx, p.ctx_off[PW_CTX_O]);     const void* x1 = at(ctx, p.ctx_off[PW_CTX_X1]);
    const void* u = at(ctx, p.ctx_off[PW_CTX_U]);     const void* lse = at(ctx, p.ctx_off[PW_CTX_LSE]);
    const void* mu1 = at(ctx, p.ctx_off[PW_CTX_MU1]); const void* r1 = at(ctx, p.ctx_off[PW_CTX_R1]);
    const void* mu2 = at(ctx, p.ctx_off[PW_CTX_MU2]); const void* r2 = at(ctx, p.ctx_off[PW_CTX_R2]);
    void* big = at(scratch, p.off_big);        // du [T,F], later dqkv [T,3d]
    void* td0 = at(scratch, p.off_td0);        // dh2, then dout, then dh1
    void* dx1 = at(scratch, p.off_td1);
    void* delta = at(scratch, p.off_delta);
    void* part = at(scratch, p.off_partials);

    void* part2 = at(scratch, p.off_partials2);
    void* part3 = at(scratch, p.off_partials3);
    void* part4 = at(scratch, p.off_partials4);
    ReduceJob jobs[4];                                   // LN2, db1, LN1, dbqkv: summed by one launch at the end

    // The weight gradients and the bias column sums hang off the dgrad chain, so they run on a
    // side stream: their CTAs fill the SMs that the last, partly filled round of a dgrad GEMM
    // leaves idle (and the HBM-bound kernels share SMs with GEMM CTAs).  Events order the two
    // streams; the side stream always rejoins before this call returns, so a captured graph sees
    // a plain fork/join.  While per-kernel profiling is on everything stays on one stream.
    cudaStream_t ax = (L->profiling || L->single_stream) ? st : L->aux;
    auto order = [&](cudaEvent_t ev, cudaStream_t from, cudaStream_t to) -> pw_status_t {
        if (from == to) return PW_OK;
        cudaError_t e = cudaEventRecord(ev, from);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(to, ev, 0);
        return e == cudaSuccess ? PW_OK : fail_cuda("stream ordering", e);
    };
    PW_DO(order(L->ev[0], st, ax));                      // side stream starts after everything already enqueued
    // Lean ctx: the three operands of the weight-gradient GEMMs that were not kept are made again on
    // the side stream, each just before the GEMM that reads it.  The statistics the LayerNorm kernel
    // writes once more go to scratch (the ctx is read-only here).
    void* lean_st1 = p.lean ? at(scratch, p.off_lean_stats) : nullptr;
    void* lean_st2 = p.lean ? at(scratch, p.off_lean_stats + align256(static_cast<size_t>(T) * 4)) : nullptr;
    if (rederive) {
        LaunchScope sc(L, PW_K_GELU, 1, 0.0, 4.0 * T * F, ax);
        const char* e = launch_gelu_fwd(L->rt, u, const_cast<void*>(a), static_cast<long long>(T) * F, act, ax);
        if (e) return fail(PW_ERR_CUDA, e);
    }
    // y = x1 + a W2^T + b2  ->  du = (dy W2) * gelu'(u),  dW2 = dy^T a
    PW_DO(do_gemm(L, gemm_args(kNT, kEpiF32, act, d, F, T, dy, d, a, F, G->w_fc2, F, nullptr, nullptr, 0,
                                     nullptr, accumulate), ax));
    void* sk = at(scratch, p.off_splitk);                // dgrad GEMMs run one after the other on the calling stream
    PW_DO(do_gemm(L, gemm_args(kNN, kEpiDGelu, act, T, F, d, dy, d, P->w_fc2, F, big, F, nullptr, u, F,
                                     nullptr, 0, sk), st));
    PW_DO(order(L->ev[1], st, ax));                      // du ready
    // u = h2 W1^T + b1  ->  dh2 = du W1,  dW1 = du^T h2,  db1 = colsum(du)
    if (rederive) PW_DO(do_ln_fwd(L, x1, P->ln2_gamma, P->ln2_beta, const_cast<void*>(h2), lean_st1, lean_st2, ax));
    PW_DO(do_gemm(L, gemm_args(kNT, kEpiF32, act, F, d, T, big, F, h2, d, G->w_fc1, d, nullptr, nullptr, 0,
                                     nullptr, accumulate), ax));
    PW_DO(do_colsum(L, big, F, G->b_fc1, accumulate, part2, ax, &jobs[1]));
    if (ax != st) {                                      // remembered: du may be overwritten only after these two
        cudaError_t e = cudaEventRecord(L->ev[2], ax);
        if (e != cudaSuccess) return fail_cuda("stream ordering", e);
    }
    PW_DO(do_gemm(L, gemm_args(kNN, kEpiNone, act, T, d, F, big, F, P->w_fc1, d, td0, d, nullptr, nullptr, 0,
                                     nullptr, 0, sk), st));
    // LN2 backward + residual: dx1 = dy + LNbwd(dh2); also db2 = colsum(dy), dbo = colsum(dx1)
    PW_DO(do_ln_bwd(L, td0, x1, mu2, r2, P->ln2_gamma, dy, dx1, G->ln2_gamma, G->ln2_beta,
                                G->b_fc2, G->b_o, accumulate, part, st, &jobs[0]));
    PW_DO(order(L->ev[3], st, ax));                      // dx1 ready
    // x1 = x + o Wo^T + bo  ->  dout = dx1 Wo,  dWo = dx1^T o
    PW_DO(do_gemm(L, gemm_args(kNT, kEpiF32, act, d, d, T, dx1, d, o, d, G->w_o, d, nullptr, nullptr, 0,
                                     nullptr, accumulate), ax));
    // (the epilogue also takes delta = rowsum(dout * o) per token and head, which attention backward starts from)
    {
        GemmArgs g = gemm_args(kNN, kEpiRowDot, act, T, d, d, dx1, d, P->w_o, d, td0, d, nullptr, o, d, nullptr, 0, sk);
        g.row_dot = delta; g.head_dim = p.dh; g.seq_len = p.S;
        PW_DO(do_gemm(L, g, st));
    }
    // attention backward -> dqkv (reuses the du buffer)
    if (ax != st) {
        cudaError_t e = cudaStreamWaitEvent(st, L->ev[2], 0);
        if (e != cudaSuccess) return fail_cuda("stream ordering", e);
    }
    PW_DO(do_attn_bwd(L, qkv, nullptr, td0, lse, big, delta, st));
    PW_DO(order(L->ev[4], st, ax));                      // dqkv ready
    // qkv = h1 Wqkv^T + bqkv  ->  dh1 = dqkv Wqkv,  dWqkv = dqkv^T h1,  dbqkv = colsum(dqkv)
    if (rederive) PW_DO(do_ln_fwd(L, x, P->ln1_gamma, P->ln1_beta, const_cast<void*>(h1), lean_st1, lean_st2, ax));
    PW_DO(do_gemm(L, gemm_args(kNT, kEpiF32, act, 3 * d, d, T, big, 3 * d, h1, d, G->w_qkv, d, nullptr, nullptr,
                                     0, nullptr, accumulate), ax));
    PW_DO(do_colsum(L, big, 3 * d, G->b_qkv, accumulate, part4, ax, &jobs[3]));
    PW_DO(do_gemm(L, gemm_args(kNN, kEpiNone, act, T, d, 3 * d, big, 3 * d, P->w_qkv, d, td0, d, nullptr,
                                     nullptr, 0, nullptr, 0, sk), st));
    // LN1 backward + residual: dx = dx1 + LNbwd(dh1)
    PW_DO(do_ln_bwd(L, td0, x, mu1, r1, P->ln1_gamma, dx1, dx, G->ln1_gamma, G->ln1_beta, nullptr,
                                nullptr, accumulate, part3, st, &jobs[2]));
    PW_DO(order(L->ev[5], ax, st));                      // join
    // dgamma1/2, dbeta1/2, db2, dbo, db1, dbqkv: eight vectors, one fixed-order launch
    PW_DO(do_reduce(L, jobs, 4, accumulate, st));
    return PW_OK;
}

static bool params_ok(const pw_layer_params_t* P)
{
    const void* const* q = reinterpret_cast<const void* const*>(P);
    for (int i = 0; i < 12; ++i)
        if (q[i] == nullptr || (reinterpret_cast<uintptr_t>(q[i]) & 15)) return false;
    return true;
}
static bool grads_ok(const pw_layer_grads_t* G)
{
    void* const* q = reinterpret_cast<void* const*>(G);
    for (int i = 0; i < 12; ++i)
        if (q[i] == nullptr || (reinterpret_cast<uintptr_t>(q[i]) & 15)) return false;
    return true;
}
static bool aligned(const void* q, size_t a) { return q != nullptr && (reinterpret_cast<uintptr_t>(q) & (a - 1)) == 0; }

static pw_status_t read_status(DeviceStatus* dev, int* code, int* site)
{
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail_cuda("cudaDeviceSynchronize", e);
    DeviceStatus h;
    e = cudaMemcpy(&h, dev, sizeof(h), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda("cudaMemcpy(status)", e);
    if (code) *code = h.code;
    if (site) *site = h.site;
    // A kernel that gave up may have left the work counters of the persistent attention kernels
    // mid-count; the device is idle here, so they are put back to zero (the error stays recorded).
    // (the same goes for the split-K tickets of the GEMM, which follow the counters in the struct)
    if (h.code != 0)
        cudaMemset(reinterpret_cast<char*>(dev) + offsetof(DeviceStatus, sched), 0, sizeof(h.sched) + sizeof(h.tickets));
    return PW_OK;
}

}  // namespace pw

using namespace pw;

extern "C" {

int pw_version(void) { return PW_VERSION; }

const char* pw_status_string(pw_status_t s)
{
    switch (s) {
        case PW_OK: return "PW_OK";
        case PW_ERR_INVALID_ARG: return "PW_ERR_INVALID_ARG";
        case PW_ERR_UNSUPPORTED_SHAPE: return "PW_ERR_UNSUPPORTED_SHAPE";
        case PW_ERR_WORKSPACE_TOO_SMALL: return "PW_ERR_WORKSPACE_TOO_SMALL";
        case PW_ERR_CUDA: return "PW_ERR_CUDA";
        case PW_ERR_DEVICE_UNSUPPORTED: return "PW_ERR_DEVICE_UNSUPPORTED";
        case PW_ERR_TIMEOUT: return "PW_ERR_TIMEOUT";
        case PW_ERR_INTERNAL: return "PW_ERR_INTERNAL";
    }
    return "PW_ERR_UNKNOWN";
}

const char* pw_last_error(void) { return g_last_error.c_str(); }

pw_status_t pw_layer_create(const pw_layer_config_t* cfg, pw_layer_t** out)
{
    if (!out) return fail(PW_ERR_INVALID_ARG, "out is NULL");
    pw_status_t s = validate_cfg(cfg);
    if (s != PW_OK) return s;
    const char* err = nullptr;
    Runtime* rt = get_runtime(&err);
    if (!rt) return fail(PW_ERR_DEVICE_UNSUPPORTED, err ? err : "runtime unavailable");
    pw_layer_t* L = new (std::nothrow) pw_layer();
    if (!L) return fail(PW_ERR_INTERNAL, "out of host memory");
    L->rt = rt;
    build_plan(*cfg, rt, &L->plan);
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&L->status), sizeof(DeviceStatus));
    if (e == cudaSuccess) e = cudaMemset(L->status, 0, sizeof(DeviceStatus));
    if (e == cudaSuccess && L->plan.whole) {
        const size_t bytes = (2 + kWholeLayerMaxTiles) * sizeof(unsigned);
        e = cudaMalloc(reinterpret_cast<void**>(&L->whole_sync), bytes);
        if (e == cudaSuccess) e = cudaMemset(L->whole_sync, 0, bytes);
    }
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&L->aux, cudaStreamNonBlocking);
    for (int i = 0; i < 6 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&L->ev[i], cudaEventDisableTiming);
    if (e != cudaSuccess) { pw_layer_destroy(L); return fail_cuda("handle resources (status word, side stream, events)", e); }
    if (log_enabled(PW_LOG_INFO)) {
        const LayerPlan& p = L->plan;
        log_line(PW_LOG_INFO, "pw_layer_create: d_model " + std::to_string(p.d) + ", " + std::to_string(p.H) + " heads x " + std::to_string(p.dh) +
                                  ", d_ff " + std::to_string(p.F) + ", " + std::to_string(p.B) + " x " + std::to_string(p.S) + " tokens, ctx " +
                                  std::to_string(p.ctx_bytes) + " bytes, scratch " + std::to_string(p.scratch_bytes) + " bytes" +
                                  (p.lean ? ", lean save set" : "") + (p.whole ? ", whole-layer kernels" : ""));
    }
    *out = L;
    return PW_OK;
}

void pw_layer_destroy(pw_layer_t* layer)
{
    if (!layer) return;
    for (auto& sp : layer->spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    for (auto e : layer->pool) cudaEventDestroy(e);
    for (auto e : layer->ev) if (e) cudaEventDestroy(e);
    if (layer->aux) cudaStreamDestroy(layer->aux);
    if (layer->status) cudaFree(layer->status);
    if (layer->whole_sync) cudaFree(layer->whole_sync);
    delete layer;
}

pw_status_t pw_layer_workspace_bytes(const pw_layer_t* layer, size_t* ctx_bytes, size_t* scratch_bytes)
{
    if (!layer) return fail(PW_ERR_INVALID_ARG, "layer is NULL");
    if (ctx_bytes) *ctx_bytes = layer->plan.ctx_bytes;
    if (scratch_bytes) *scratch_bytes = layer->plan.scratch_bytes;
    return PW_OK;
}

pw_status_t pw_layer_ctx_offset(const pw_layer_t* layer, int which, size_t* offset, size_t* bytes)
{
    if (!layer || which < 0 || which >= PW_CTX_COUNT) return fail(PW_ERR_INVALID_ARG, "bad layer or tensor id");
    if (offset) *offset = layer->plan.ctx_off[which];
    if (bytes) *bytes = layer->plan.ctx_size[which];
    return PW_OK;
}

pw_status_t pw_layer_fwd(pw_layer_t* layer, const pw_layer_params_t* params, const void* x, void* y, void* ctx,
                         void* scratch, void* stream)
{
    NvtxRange nv("pw_layer_fwd");
    if (!layer || !params) return fail(PW_ERR_INVALID_ARG, "layer or params is NULL");
    if (!params_ok(params)) return fail(PW_ERR_INVALID_ARG, "a parameter pointer is NULL or not 16-byte aligned");
    if (!aligned(x, 16) || !aligned(y, 16)) return fail(PW_ERR_INVALID_ARG, "x or y is NULL or misaligned");
    if (x == y) return fail(PW_ERR_INVALID_ARG, "y must not alias x");
    if (ctx == nullptr && !aligned(scratch, 256)) return fail(PW_ERR_INVALID_ARG, "scratch must be 256-byte aligned when ctx is NULL");
    if (ctx != nullptr && !aligned(ctx, 256)) return fail(PW_ERR_INVALID_ARG, "ctx must be 256-byte aligned");
    if (layer->plan.lean && !aligned(scratch, 256)) return fail(PW_ERR_INVALID_ARG, "a lean-ctx layer needs a 256-byte aligned scratch in fwd");
    if (layer->plan.whole && !aligned(scratch, 256)) return fail(PW_ERR_INVALID_ARG, "a whole-layer handle needs a 256-byte aligned scratch in fwd");
    return enqueue_fwd(layer, params, x, y, ctx ? ctx : scratch, scratch, true, static_cast<cudaStream_t>(stream));
}

pw_status_t pw_layer_bwd(pw_layer_t* layer, const pw_layer_params_t* params, const void* x, const void* dy, void* dx,
                         const pw_layer_grads_t* grads, int accumulate, const void* ctx, void* scratch, void* stream)
{
    NvtxRange nv("pw_layer_bwd");
    if (!layer || !params || !grads) return fail(PW_ERR_INVALID_ARG, "layer, params or grads is NULL");
    if (!params_ok(params)) return fail(PW_ERR_INVALID_ARG, "a parameter pointer is NULL or not 16-byte aligned");
    if (!grads_ok(grads)) return fail(PW_ERR_INVALID_ARG, "a gradient pointer is NULL or not 16-byte aligned");
    if (!aligned(x, 16) || !aligned(dy, 16) || !aligned(dx, 16)) return fail(PW_ERR_INVALID_ARG, "x, dy or dx is NULL or misaligned");
    if (dx == x) return fail(PW_ERR_INVALID_ARG, "dx must not alias x");
    if (!aligned(scratch, 256)) return fail(PW_ERR_INVALID_ARG, "scratch is NULL or not 256-byte aligned");
    if (ctx != nullptr && !aligned(ctx, 256)) return fail(PW_ERR_INVALID_ARG, "ctx must be 256-byte aligned");
    if (accumulate != 0 && accumulate != 1) return fail(PW_ERR_INVALID_ARG, "accumulate must be 0 or 1");
    return enqueue_bwd(layer, params, x, dy, dx, grads, accumulate, ctx, scratch, static_cast<cudaStream_t>(stream));
}

pw_status_t pw_layer_status(pw_layer_t* layer, int* device_status, int* site)
{
    if (!layer) return fail(PW_ERR_INVALID_ARG, "layer is NULL");
    return read_status(layer->status, device_status, site);
}

pw_status_t pw_layer_profile_begin(pw_layer_t* layer)
{
    if (!layer) return fail(PW_ERR_INVALID_ARG, "layer is NULL");
    for (auto& sp : layer->spans) { layer->pool.push_back(sp.a); layer->pool.push_back(sp.b); }
    layer->spans.clear();
    std::memset(&layer->prof, 0, sizeof(layer->prof));
    layer->profiling = true;
    return PW_OK;
}

pw_status_t pw_layer_profile_end(pw_layer_t* layer, pw_profile_t* out)
{
    if (!layer || !out) return fail(PW_ERR_INVALID_ARG, "layer or out is NULL");
    if (!layer->profiling) return fail(PW_ERR_INVALID_ARG, "profile_end without profile_begin");
    layer->profiling = false;
    cudaError_t e = cudaStreamSynchronize(layer->prof_stream);
    if (e != cudaSuccess) return fail_cuda("cudaStreamSynchronize", e);
    for (auto& sp : layer->spans) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, sp.a, sp.b) == cudaSuccess) layer->prof.ms[sp.cls] += ms;
        layer->pool.push_back(sp.a); layer->pool.push_back(sp.b);
    }
    layer->spans.clear();
    *out = layer->prof;
    return PW_OK;
}

pw_status_t pw_layer_launch_count(const pw_layer_t* layer, uint64_t* count)
{
    if (!layer || !count) return fail(PW_ERR_INVALID_ARG, "layer or count is NULL");
    *count = layer->launches;
    return PW_OK;
}

// ---------------------------------------------------------------------------------------- stage

pw_status_t pw_stage_create(const pw_layer_config_t* cfg, int n_layers, pw_stage_t** out)
{
    if (!out) return fail(PW_ERR_INVALID_ARG, "out is NULL");
    if (n_layers <= 0 || n_layers > 4096) return fail(PW_ERR_INVALID_ARG, "n_layers out of range");
    pw_layer_t* L = nullptr;
    pw_status_t s = pw_layer_create(cfg, &L);
    if (s != PW_OK) return s;
    pw_stage_t* st = new (std::nothrow) pw_stage();
    if (!st) { pw_layer_destroy(L); return fail(PW_ERR_INTERNAL, "out of host memory"); }
    st->layer = L;
    st->n_layers = n_layers;
    *out = st;
    if (log_enabled(PW_LOG_INFO)) log_line(PW_LOG_INFO, "pw_stage_create: " + std::to_string(n_layers) + " layers of the shape above");
    return PW_OK;
}

void pw_stage_destroy(pw_stage_t* stage)
{
    if (!stage) return;
    for (auto& kv : stage->graphs) cudaGraphExecDestroy(kv.second.exec);
    pw_layer_destroy(stage->layer);
    delete stage;
}

namespace {
struct StageLayout {
    size_t act_bytes, n_act;      // hand-off buffers [T,d] bf16 between layers
    size_t ctx_bytes, n_ctx;      // saved contexts (recompute == 0)
    size_t off_act, off_ctx, off_g0, off_g1, off_scratch, total;
};
pw_status_t stage_layout(const pw_stage_t* stage, int M, int schedule, int recompute, StageLayout* lay)
{
    if (M <= 0 || M > 65536) return fail(PW_ERR_INVALID_ARG, "n_microbatches out of range");
    if (schedule != PW_SCHEDULE_GPIPE && schedule != PW_SCHEDULE_PER_MICROBATCH) return fail(PW_ERR_INVALID_ARG, "unknown schedule");
    if (recompute != 0 && recompute != 1) return fail(PW_ERR_INVALID_ARG, "recompute must be 0 or 1");
    const LayerPlan& p = stage->layer->plan;
    const size_t L = stage->n_layers, live = (schedule == PW_SCHEDULE_GPIPE) ? M : 1;
    lay->act_bytes = align256(static_cast<size_t>(p.T) * p.d * 2);
    lay->n_act = (L - 1) * live;
    lay->ctx_bytes = p.ctx_bytes;
    lay->n_ctx = recompute ? 0 : L * live;
    size_t s = 0;
    lay->off_act = s; s += lay->act_bytes * lay->n_act;
    lay->off_ctx = s; s += lay->ctx_bytes * lay->n_ctx;
    lay->off_g0 = s; s += lay->act_bytes;
    lay->off_g1 = s; s += lay->act_bytes;
    lay->off_scratch = s; s += p.scratch_bytes;
    lay->total = s;
    return PW_OK;
}
}  // namespace

pw_status_t pw_stage_workspace_bytes(const pw_stage_t* stage, int n_microbatches, int schedule, int recompute,
                                     size_t* bytes)
{
    if (!stage || !bytes) return fail(PW_ERR_INVALID_ARG, "stage or bytes is NULL");
    StageLayout lay;
    pw_status_t s = stage_layout(stage, n_microbatches, schedule, recompute, &lay);
    if (s != PW_OK) return s;
    *bytes = lay.total;
    return PW_OK;
}

namespace {
// Enqueues the whole chain on `st`.  sync_each = OPBYOP.
pw_status_t enqueue_chain(pw_stage_t* stage, const pw_layer_params_t* params, const pw_layer_grads_t* grads,
                          const void* const* x_mb, const void* const* dy_mb, void* const* y_mb, void* const* dx_mb,
                          int M, int schedule, int recompute, void* ws, const StageLayout& lay, bool sync_each,
                          cudaStream_t st)
{
    pw_layer_t* Lh = stage->layer;
    const int L = stage->n_layers;
    const bool gpipe = schedule == PW_SCHEDULE_GPIPE;
    auto act = [&](int m, int l) -> void* {   // input of layer l (l >= 1) for micro-batch m
        const size_t slot = (gpipe ? static_cast<size_t>(m) * (L - 1) : 0) + (l - 1);
        return at(ws, lay.off_act + slot * lay.act_bytes);
    };
    auto ctxp = [&](int m, int l) -> void* {
        if (recompute) return nullptr;
        const size_t slot = (gpipe ? static_cast<size_t>(m) * L : 0) + l;
        return at(ws, lay.off_ctx + slot * lay.ctx_bytes);
    };
    void* scratch = at(ws, lay.off_scratch);
    auto sync = [&]() -> pw_status_t {
        if (!sync_each) return PW_OK;
        cudaError_t e = cudaStreamSynchronize(st);
        return e == cudaSuccess ? PW_OK : fail_cuda("cudaStreamSynchronize", e);
    };
    auto fwd_mb = [&](int m) -> pw_status_t {
        for (int l = 0; l < L; ++l) {
            const void* in = l == 0 ? x_mb[m] : act(m, l);
            void* out = l == L - 1 ? y_mb[m] : act(m, l + 1);
            void* c = ctxp(m, l);
            pw_status_t s = enqueue_fwd(Lh, &params[l], in, out, c ? c : scratch, scratch, true, st);
            if (s != PW_OK) return s;
            if ((s = sync()) != PW_OK) return s;
        }
        return PW_OK;
    };
    auto bwd_mb = [&](int m) -> pw_status_t {
        const void* g = dy_mb[m];
        for (int l = L - 1; l >= 0; --l) {
            const void* in = l == 0 ? x_mb[m] : act(m, l);
            void* out = l == 0 ? dx_mb[m] : at(ws, (l & 1) ? lay.off_g1 : lay.off_g0);
            pw_status_t s = enqueue_bwd(Lh, &params[l], in, g, out, &grads[l], m > 0 ? 1 : 0, ctxp(m, l), scratch, st);
            if (s != PW_OK) return s;
            if ((s = sync()) != PW_OK) return s;
            g = out;
        }
        return PW_OK;
    };
    pw_status_t s;
    if (gpipe) {
        for (int m = 0; m < M; ++m) if ((s = fwd_mb(m)) != PW_OK) return s;
        for (int m = 0; m < M; ++m) if ((s = bwd_mb(m)) != PW_OK) return s;
    } else {
        for (int m = 0; m < M; ++m) {
            if ((s = fwd_mb(m)) != PW_OK) return s;
            if ((s = bwd_mb(m)) != PW_OK) return s;
        }
    }
    return PW_OK;
}
}  // namespace

pw_status_t pw_stage_run_chain(pw_stage_t* stage, const pw_layer_params_t* params, const pw_layer_grads_t* grads,
                               const void* const* x_mb, const void* const* dy_mb, void* const* y_mb,
                               void* const* dx_mb, int n_microbatches, int dispatch_mode, int schedule, int recompute,
                               void* workspace, size_t workspace_bytes, void* stream)
{
    NvtxRange nv("pw_stage_run_chain");
    if (!stage || !params || !grads || !x_mb || !dy_mb || !y_mb || !dx_mb)
        return fail(PW_ERR_INVALID_ARG, "a required pointer is NULL");
    if (dispatch_mode < PW_DISPATCH_OPBYOP || dispatch_mode > PW_DISPATCH_GRAPH) return fail(PW_ERR_INVALID_ARG, "unknown dispatch mode");
    StageLayout lay;
    pw_status_t s = stage_layout(stage, n_microbatches, schedule, recompute, &lay);
    if (s == PW_OK && log_enabled(PW_LOG_INFO))
        log_line(PW_LOG_INFO, std::string("pw_stage_run_chain: ") + (dispatch_mode == PW_DISPATCH_OPBYOP ? "OPBYOP" : dispatch_mode == PW_DISPATCH_ASYNC ? "ASYNC" : "GRAPH") +
                                  ", " + std::to_string(stage->n_layers) + " layers x " + std::to_string(n_microbatches) + " micro-batches" + (recompute ? ", recompute" : ""));
    if (s != PW_OK) return s;
    if (!aligned(workspace, 256)) return fail(PW_ERR_INVALID_ARG, "workspace is NULL or not 256-byte aligned");
    if (workspace_bytes < lay.total) return fail(PW_ERR_WORKSPACE_TOO_SMALL, "workspace smaller than pw_stage_workspace_bytes reports");
    const int L = stage->n_layers, M = n_microbatches;
    for (int l = 0; l < L; ++l)
        if (!params_ok(&params[l]) || !grads_ok(&grads[l])) return fail(PW_ERR_INVALID_ARG, "a parameter or gradient pointer is NULL or misaligned");
    for (int m = 0; m < M; ++m) {
        if (!aligned(x_mb[m], 16) || !aligned(dy_mb[m], 16) || !aligned(y_mb[m], 16) || !aligned(dx_mb[m], 16))
            return fail(PW_ERR_INVALID_ARG, "a micro-batch pointer is NULL or misaligned");
        if (x_mb[m] == y_mb[m] || x_mb[m] == dx_mb[m]) return fail(PW_ERR_INVALID_ARG, "y and dx must not alias x");
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    if (dispatch_mode != PW_DISPATCH_GRAPH)
        return enqueue_chain(stage, params, grads, x_mb, dy_mb, y_mb, dx_mb, M, schedule, recompute, workspace, lay,
                             dispatch_mode == PW_DISPATCH_OPBYOP, st);

    // GRAPH: key = every pointer and setting that the captured launches bake in.
    std::vector<uint64_t> key;
    key.reserve(8 + 24 * L + 4 * M);
    key.push_back(M); key.push_back(schedule); key.push_back(recompute); key.push_back(stage->layer->single_stream ? 1 : 0);
    key.push_back(tuning().epoch);
    key.push_back(reinterpret_cast<uint64_t>(workspace));
    for (int l = 0; l < L; ++l) {
        const void* const* pp = reinterpret_cast<const void* const*>(&params[l]);
        void* const* gg = reinterpret_cast<void* const*>(&grads[l]);
        for (int i = 0; i < 12; ++i) { key.push_back(reinterpret_cast<uint64_t>(pp[i])); key.push_back(reinterpret_cast<uint64_t>(gg[i])); }
    }
    for (int m = 0; m < M; ++m) {
        key.push_back(reinterpret_cast<uint64_t>(x_mb[m])); key.push_back(reinterpret_cast<uint64_t>(dy_mb[m]));
        key.push_back(reinterpret_cast<uint64_t>(y_mb[m])); key.push_back(reinterpret_cast<uint64_t>(dx_mb[m]));
    }
    if (stage->layer->profiling) return fail(PW_ERR_INVALID_ARG, "per-kernel profiling is not available in GRAPH mode");
    auto it = stage->graphs.find(key);
    if (it == stage->graphs.end()) {
        if (st == nullptr) return fail(PW_ERR_INVALID_ARG, "GRAPH mode needs a non-default stream (the legacy stream cannot be captured)");
        cudaError_t e = cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal);
        if (e != cudaSuccess) return fail_cuda("cudaStreamBeginCapture", e);
        stage->layer->capturing = true;
        stage->layer->graph_nodes = 0;
        s = enqueue_chain(stage, params, grads, x_mb, dy_mb, y_mb, dx_mb, M, schedule, recompute, workspace, lay, false, st);
        stage->layer->capturing = false;
        cudaGraph_t graph = nullptr;
        e = cudaStreamEndCapture(st, &graph);
        if (s != PW_OK) { if (graph) cudaGraphDestroy(graph); return s; }
        if (e != cudaSuccess) return fail_cuda("cudaStreamEndCapture", e);
        cudaGraphExec_t exec = nullptr;
        e = cudaGraphInstantiate(&exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) return fail_cuda("cudaGraphInstantiate", e);
        if (stage->graphs.size() >= 16) {   // bounded cache
            for (auto& kv : stage->graphs) cudaGraphExecDestroy(kv.second.exec);
            stage->graphs.clear();
        }
        it = stage->graphs.emplace(key, pw_stage::Cached{exec, stage->layer->graph_nodes}).first;
    }
    cudaError_t e = cudaGraphLaunch(it->second.exec, st);
    if (e != cudaSuccess) return fail_cuda("cudaGraphLaunch", e);
    stage->layer->launches += it->second.nodes;
    return PW_OK;
}

pw_status_t pw_stage_status(pw_stage_t* stage, int* device_status, int* site)
{
    if (!stage) return fail(PW_ERR_INVALID_ARG, "stage is NULL");
    return read_status(stage->layer->status, device_status, site);
}
pw_status_t pw_stage_profile_begin(pw_stage_t* stage)
{
    if (!stage) return fail(PW_ERR_INVALID_ARG, "stage is NULL");
    return pw_layer_profile_begin(stage->layer);
}
pw_status_t pw_stage_profile_end(pw_stage_t* stage, pw_profile_t* out)
{
    if (!stage) return fail(PW_ERR_INVALID_ARG, "stage is NULL");
    return pw_layer_profile_end(stage->layer, out);
}
pw_status_t pw_stage_launch_count(const pw_stage_t* stage, uint64_t* count)
{
    if (!stage) return fail(PW_ERR_INVALID_ARG, "stage is NULL");
    return pw_layer_launch_count(stage->layer, count);
}

pw_status_t pw_layer_set_side_stream(pw_layer_t* layer, int enabled)
{
    if (!layer) return fail(PW_ERR_INVALID_ARG, "layer is NULL");
    layer->single_stream = enabled == 0;
    return PW_OK;
}
pw_status_t pw_stage_set_side_stream(pw_stage_t* stage, int enabled)
{
    if (!stage) return fail(PW_ERR_INVALID_ARG, "stage is NULL");
    return pw_layer_set_side_stream(stage->layer, enabled);
}

// ---------------------------------------------------------------------------------------- language model step
namespace {
struct LmLayout {
    size_t act_bytes, off_x0, off_acts, off_ctx, off_hf, off_mu, off_r, off_logits, off_lse, off_rows, off_g0, off_g1,
        off_emb, off_scratch, total;
};
pw_status_t lm_layout(const pw_stage_t* stage, int vocab, int recompute, LmLayout* lay)
{
    if (vocab <= 0 || (vocab % 8)) return fail(PW_ERR_UNSUPPORTED_SHAPE, "vocab must be a positive multiple of 8");
    if (recompute != 0 && recompute != 1) return fail(PW_ERR_INVALID_ARG, "recompute must be 0 or 1");
    const LayerPlan& p = stage->layer->plan;
    const size_t L = stage->n_layers, T = p.T;
    lay->act_bytes = align256(T * p.d * 2);
    size_t s = 0;
    lay->off_x0 = s; s += lay->act_bytes;
    lay->off_acts = s; s += lay->act_bytes * L;                 // output of every layer (the last one feeds the final LayerNorm)
    lay->off_ctx = s; s += recompute ? 0 : p.ctx_bytes * L;
    lay->off_hf = s; s += lay->act_bytes;
    lay->off_mu = s; s += align256(T * 4);
    lay->off_r = s; s += align256(T * 4);
    lay->off_logits = s; s += align256(T * static_cast<size_t>(vocab) * 2);
    lay->off_lse = s; s += align256(T * 4);
    lay->off_rows = s; s += align256(T * 4);
    lay->off_g0 = s; s += lay->act_bytes;
    lay->off_g1 = s; s += lay->act_bytes;
    lay->off_emb = s; s += align256(embedding_bwd_scratch_bytes(static_cast<int>(T), vocab));
    lay->off_scratch = s; s += p.scratch_bytes;
    lay->total = s;
    return PW_OK;
}
}  // namespace

pw_status_t pw_lm_workspace_bytes(const pw_stage_t* stage, int vocab, int recompute, size_t* bytes)
{
    if (!stage || !bytes) return fail(PW_ERR_INVALID_ARG, "stage or bytes is NULL");
    LmLayout lay;
    pw_status_t s = lm_layout(stage, vocab, recompute, &lay);
    if (s != PW_OK) return s;
    *bytes = lay.total;
    return PW_OK;
}

pw_status_t pw_lm_step(pw_stage_t* stage, const pw_layer_params_t* params, const pw_layer_grads_t* grads,
                       const pw_lm_params_t* lm, const pw_lm_grads_t* lm_grads, const int32_t* ids, const int32_t* labels,
                       float* loss, int vocab, int recompute, void* workspace, size_t workspace_bytes, void* stream)
{
    NvtxRange nv("pw_lm_step");
    if (!stage || !params || !grads || !lm || !lm_grads || !ids || !labels || !loss)
        return fail(PW_ERR_INVALID_ARG, "a required pointer is NULL");
    LmLayout lay;
    pw_status_t s = lm_layout(stage, vocab, recompute, &lay);
    if (s != PW_OK) return s;
    if (!aligned(workspace, 256)) return fail(PW_ERR_INVALID_ARG, "workspace is NULL or not 256-byte aligned");
    if (workspace_bytes < lay.total) return fail(PW_ERR_WORKSPACE_TOO_SMALL, "workspace smaller than pw_lm_workspace_bytes reports");
    pw_layer_t* Lh = stage->layer;
    const LayerPlan& p = Lh->plan;
    const int L = stage->n_layers, T = p.T, d = p.d, V = vocab;
    for (int l = 0; l < L; ++l)
        if (!params_ok(&params[l]) || !grads_ok(&grads[l])) return fail(PW_ERR_INVALID_ARG, "a parameter or gradient pointer is NULL or misaligned");
    if (!aligned(lm->embedding, 16) || !aligned(lm->lnf_gamma, 16) || !aligned(lm->lnf_beta, 16) ||
        !aligned(lm_grads->embedding, 16) || !aligned(lm_grads->lnf_gamma, 16) || !aligned(lm_grads->lnf_beta, 16) ||
        !aligned(ids, 4) || !aligned(labels, 4) || !aligned(loss, 4))
        return fail(PW_ERR_INVALID_ARG, "a language-model pointer is NULL or misaligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* ws = workspace;
    void* x0 = at(ws, lay.off_x0);
    auto actp = [&](int l) -> void* { return at(ws, lay.off_acts + static_cast<size_t>(l) * lay.act_bytes); };   // output of layer l
    auto ctxp = [&](int l) -> void* { return recompute ? nullptr : at(ws, lay.off_ctx + static_cast<size_t>(l) * p.ctx_bytes); };
    void* scratch = at(ws, lay.off_scratch);
    void* hf = at(ws, lay.off_hf); void* mu = at(ws, lay.off_mu); void* r = at(ws, lay.off_r);
    void* logits = at(ws, lay.off_logits); void* lse = at(ws, lay.off_lse); void* rows = at(ws, lay.off_rows);
    const char* e;

    // forward: lookup, L layers, final LayerNorm, tied projection, softmax / cross-entropy
    {
        LaunchScope sc(Lh, PW_K_EMBED, 1, 0.0, 4.0 * T * d, st);
        if ((e = launch_embedding_fwd(Lh->rt, ids, lm->embedding, T, d, V, x0, Lh->status, st))) return fail(PW_ERR_CUDA, e);
    }
    for (int l = 0; l < L; ++l) {
        void* c = ctxp(l);
        PW_DO(enqueue_fwd(Lh, &params[l], l == 0 ? x0 : actp(l - 1), actp(l), c ? c : scratch, scratch, true, st));
    }
    const void* hL = L > 0 ? actp(L - 1) : x0;
    PW_DO(do_ln_fwd(Lh, hL, lm->lnf_gamma, lm->lnf_beta, hf, mu, r, st));
    PW_DO(do_gemm(Lh, gemm_args(kTN, kEpiNone, 0, T, V, d, hf, d, lm->embedding, d, logits, V, nullptr, nullptr, 0,
                                      nullptr, 0), st));
    {
        LaunchScope sc(Lh, PW_K_XENT, 2, 0.0, 4.0 * T * V + 12.0 * T, st);
        if ((e = launch_softmax_xent(Lh->rt, logits, V, labels, T, V, 1.0f / static_cast<float>(T), lse, rows, Lh->status, st)))
            return fail(PW_ERR_CUDA, e);
        if ((e = launch_sum_scale(rows, T, 1.0f / static_cast<float>(T), loss, st))) return fail(PW_ERR_CUDA, e);
    }
    // backward: dhf = dz E, dE = dz^T hf, final LayerNorm, L layers, scatter-add of the input gradient
    void* g0 = at(ws, lay.off_g0); void* g1 = at(ws, lay.off_g1);
    PW_DO(do_gemm(Lh, gemm_args(kNN, kEpiNone, 0, T, d, V, logits, V, lm->embedding, d, g0, d, nullptr, nullptr, 0,
                                      nullptr, 0), st));
    PW_DO(do_gemm(Lh, gemm_args(kNT, kEpiF32, 0, V, d, T, logits, V, hf, d, lm_grads->embedding, d, nullptr, nullptr, 0,
                                      nullptr, 0), st));
    PW_DO(do_ln_bwd(Lh, g0, hL, mu, r, lm->lnf_gamma, nullptr, g1, lm_grads->lnf_gamma, lm_grads->lnf_beta, nullptr,
                          nullptr, 0, at(scratch, p.off_partials), st));
    const void* g = g1;
    for (int l = L - 1; l >= 0; --l) {
        void* out = (g == g1) ? g0 : g1;
        PW_DO(enqueue_bwd(Lh, &params[l], l == 0 ? x0 : actp(l - 1), g, out, &grads[l], 0, ctxp(l), scratch, st));
        g = out;
    }
    {
        LaunchScope sc(Lh, PW_K_EMBED, 2, 0.0, 2.0 * T * d + 4.0 * (T + V), st);
        if ((e = launch_embedding_bwd(Lh->rt, ids, g, T, d, V, lm_grads->embedding, at(ws, lay.off_emb), Lh->status, st)))
            return fail(PW_ERR_CUDA, e);
    }
    return PW_OK;
}

// ---------------------------------------------------------------------------------------- single steps

#define PW_RT_OR_FAIL()                                                                       \
    const char* rt_err__ = nullptr;                                                           \
    Runtime* rt = get_runtime(&rt_err__);                                                     \
    if (!rt) return fail(PW_ERR_DEVICE_UNSUPPORTED, rt_err__ ? rt_err__ : "runtime unavailable")

#define PW_OP(expr)                                          \
    do {                                                     \
        const char* e__ = (expr);                            \
        if (e__) return fail(PW_ERR_INVALID_ARG, e__);       \
    } while (0)

pw_status_t pw_op_layernorm_fwd(const void* x, const void* gamma, const void* beta, int T, int d, float eps, void* h,
                                void* mu, void* rstd, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(x, 16) || !aligned(gamma, 16) || !aligned(beta, 16) || !aligned(h, 16) || !mu || !rstd)
        return fail(PW_ERR_INVALID_ARG, "layernorm: NULL or misaligned pointer");
    PW_OP(launch_layernorm_fwd(rt, x, gamma, beta, T, d, eps, h, mu, rstd, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

size_t pw_op_layernorm_bwd_scratch_bytes(int T, int d)
{
    const char* err = nullptr;
    Runtime* rt = get_runtime(&err);
    return rt ? layernorm_bwd_scratch_bytes(rt, T, d) : 0;
}

pw_status_t pw_op_layernorm_bwd(const void* dh, const void* x, const void* mu, const void* rstd, const void* gamma,
                                const void* resid, int T, int d, void* dx, void* dgamma, void* dbeta, void* db_resid,
                                void* db_dx, int accumulate, void* partials, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(dh, 16) || !aligned(x, 16) || !aligned(gamma, 16) || !aligned(resid, 16) || !aligned(dx, 16) || !mu ||
        !rstd || !dgamma || !dbeta || !aligned(partials, 16))
        return fail(PW_ERR_INVALID_ARG, "layernorm bwd: NULL or misaligned pointer");
    PW_OP(launch_layernorm_bwd(rt, dh, x, mu, rstd, gamma, resid, T, d, dx, dgamma, dbeta, db_resid, db_dx, accumulate,
                               partials, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

size_t pw_op_colsum_scratch_bytes(int T, int N)
{
    const char* err = nullptr;
    Runtime* rt = get_runtime(&err);
    return rt ? colsum_scratch_bytes(rt, T, N) : 0;
}

pw_status_t pw_op_colsum(const void* in, int T, int N, int ld, void* out, int accumulate, void* partials, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(in, 16) || !out || !aligned(partials, 16)) return fail(PW_ERR_INVALID_ARG, "colsum: NULL or misaligned pointer");
    PW_OP(launch_colsum(rt, in, T, N, ld, out, accumulate, partials, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_op_colsum_noalloc(const void* in, int T, int N, int ld, void* out, int accumulate, void* stream)
{
    if (!aligned(in, 16) || !out) return fail(PW_ERR_INVALID_ARG, "colsum: NULL or misaligned pointer");
    if (accumulate != 0 && accumulate != 1) return fail(PW_ERR_INVALID_ARG, "accumulate must be 0 or 1");
    if (N > 0 && static_cast<size_t>(N) > colsum_noalloc_max_columns())
        return fail(PW_ERR_WORKSPACE_TOO_SMALL, "colsum (no-allocation variant): N exceeds the 262144 columns the built-in scratch can hold");
    int kind = kErrArgument;
    const char* e = launch_colsum_noalloc(in, T, N, ld, out, accumulate, static_cast<cudaStream_t>(stream), &kind);
    if (e) return fail(kind == kErrDevice ? PW_ERR_DEVICE_UNSUPPORTED : kind == kErrCuda ? PW_ERR_CUDA : PW_ERR_INVALID_ARG, e);
    return PW_OK;
}

pw_status_t pw_op_gemm(int layout, int epilogue, int act, int M, int N, int K, const void* A, int lda, const void* B,
                       int ldb, void* C, int ldc, const void* bias, const void* aux_in, int ld_aux, void* aux_out,
                       int accumulate, void* stream)
{
    PW_RT_OR_FAIL();
    // The single-step calls share one status word and run one at a time, so this GEMM may cut the
    // tiles of a thin last round along K (scratch allocated with the runtime, never on this path).
    PW_OP(launch_gemm(rt, gemm_args(layout, epilogue, act, M, N, K, A, lda, B, ldb, C, ldc, bias, aux_in, ld_aux,
                                    aux_out, accumulate, rt->split_ws), rt->op_status, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_op_gemm_rowdot(int M, int N, int K, const void* A, int lda, const void* B, int ldb, void* C, int ldc,
                              const void* other, int ld_other, int head_dim, int seq_len, void* row_dot, void* stream)
{
    PW_RT_OR_FAIL();
    GemmArgs g = gemm_args(kNN, kEpiRowDot, 0, M, N, K, A, lda, B, ldb, C, ldc, nullptr, other, ld_other, nullptr, 0, rt->split_ws);
    g.row_dot = row_dot; g.head_dim = head_dim; g.seq_len = seq_len;
    PW_OP(launch_gemm(rt, g, rt->op_status, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_op_attention_fwd(const void* qkv, int B, int S, int H, int dh, void* o, void* lse, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(qkv, 16) || !aligned(o, 16) || !lse) return fail(PW_ERR_INVALID_ARG, "attention: NULL or misaligned pointer");
    PW_OP(launch_attention_fwd(rt, qkv, B, S, H, dh, o, lse, rt->op_status, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_op_attention_bwd(const void* qkv, const void* o, const void* dout, const void* lse, int B, int S, int H,
                                int dh, void* dqkv, void* delta, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(qkv, 16) || (o && !aligned(o, 16)) || !aligned(dout, 16) || !lse || !aligned(dqkv, 16) || !delta)
        return fail(PW_ERR_INVALID_ARG, "attention bwd: NULL or misaligned pointer");
    PW_OP(launch_attention_bwd(rt, qkv, o, dout, lse, B, S, H, dh, dqkv, delta, rt->op_status, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_op_embedding_fwd(const int32_t* ids, const void* E, int T, int d, int V, void* x0, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(ids, 4) || !aligned(E, 16) || !aligned(x0, 16)) return fail(PW_ERR_INVALID_ARG, "embedding: NULL or misaligned pointer");
    PW_OP(launch_embedding_fwd(rt, ids, E, T, d, V, x0, rt->op_status, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

size_t pw_op_embedding_bwd_scratch_bytes(int T, int V) { return embedding_bwd_scratch_bytes(T, V); }

pw_status_t pw_op_embedding_bwd(const int32_t* ids, const void* dx0, int T, int d, int V, void* dE, void* scratch,
                                void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(ids, 4) || !aligned(dx0, 16) || !aligned(dE, 16) || !aligned(scratch, 4))
        return fail(PW_ERR_INVALID_ARG, "embedding bwd: NULL or misaligned pointer");
    PW_OP(launch_embedding_bwd(rt, ids, dx0, T, d, V, dE, scratch, rt->op_status, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_op_softmax_xent(void* logits, int ld, const int32_t* labels, int T, int V, float grad_scale, void* lse,
                               void* loss_rows, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(logits, 16) || !aligned(labels, 4) || !aligned(lse, 4) || !aligned(loss_rows, 4))
        return fail(PW_ERR_INVALID_ARG, "softmax-xent: NULL or misaligned pointer");
    PW_OP(launch_softmax_xent(rt, logits, ld, labels, T, V, grad_scale, lse, loss_rows, rt->op_status,
                              static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_op_affine_f32(const void* x, long long n, float scale, float shift, void* y, void* stream)
{
    PW_RT_OR_FAIL();
    if (!aligned(x, 4) || !aligned(y, 4)) return fail(PW_ERR_INVALID_ARG, "affine: NULL or misaligned pointer");
    PW_OP(launch_affine_f32(x, n, scale, shift, y, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_sgd_apply(const pw_apply_item_t* items, int n_items, float lr, float grad_scale, int init_master,
                         void* stream)
{
    NvtxRange nv("pw_sgd_apply");
    PW_RT_OR_FAIL();
    if (!items || n_items <= 0) return fail(PW_ERR_INVALID_ARG, "gradient apply: no items");
    if (!(lr >= 0.0f) || !(grad_scale > 0.0f) || !std::isfinite(lr) || !std::isfinite(grad_scale))
        return fail(PW_ERR_INVALID_ARG, "gradient apply: lr must be finite and >= 0, grad_scale finite and > 0");
    std::vector<ApplyItem> v(static_cast<size_t>(n_items));
    for (int i = 0; i < n_items; ++i) {
        const pw_apply_item_t& a = items[i];
        if (a.n < 0) return fail(PW_ERR_INVALID_ARG, "gradient apply: negative element count");
        if (a.n > 0 && (!aligned(a.param, 2) || !aligned(a.master, 4) || !aligned(a.grad, 4)))
            return fail(PW_ERR_INVALID_ARG, "gradient apply: NULL or misaligned pointer");
        v[static_cast<size_t>(i)] = ApplyItem{a.param, a.master, a.grad, static_cast<long long>(a.n)};
    }
    PW_OP(launch_sgd_apply(v.data(), n_items, lr * grad_scale, init_master, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

pw_status_t pw_dp_slice(int64_t n_total, int world, int rank, int64_t* lo, int64_t* hi)
{
    if (n_total < 0 || world < 1 || world > kDpMaxWorld || rank < 0 || rank >= world || !lo || !hi)
        return fail(PW_ERR_INVALID_ARG, "dp slice: need n_total >= 0, 1 <= world <= 8, 0 <= rank < world, non-NULL outputs");
    long long a, b;
    dp_slice(static_cast<long long>(n_total), world, rank, &a, &b);
    *lo = a; *hi = b;
    return PW_OK;
}

pw_status_t pw_dp_reduce_apply(int rank, int world, const void* const* grads, void* const* params, void* master_slice,
                               int64_t n_total, float lr, float grad_scale, int init_master, void* stream)
{
    PW_RT_OR_FAIL();
    if (world < 1 || world > kDpMaxWorld || rank < 0 || rank >= world)
        return fail(PW_ERR_INVALID_ARG, "data-parallel apply: need 1 <= world <= 8 and 0 <= rank < world");
    if (!grads || !params || n_total < 0) return fail(PW_ERR_INVALID_ARG, "data-parallel apply: NULL pointer table or negative size");
    if (!(lr >= 0.0f) || !(grad_scale > 0.0f) || !std::isfinite(lr) || !std::isfinite(grad_scale))
        return fail(PW_ERR_INVALID_ARG, "data-parallel apply: lr must be finite and >= 0, grad_scale finite and > 0");
    for (int k = 0; k < world; ++k)
        if (!aligned(grads[k], 4) || !aligned(params[k], 2))
            return fail(PW_ERR_INVALID_ARG, "data-parallel apply: NULL or misaligned replica buffer");
    long long lo, hi;
    dp_slice(static_cast<long long>(n_total), world, rank, &lo, &hi);
    if (hi > lo && !aligned(master_slice, 4)) return fail(PW_ERR_INVALID_ARG, "data-parallel apply: NULL or misaligned master slice");
    PW_OP(launch_dp_reduce_apply(rank, world, grads, params, master_slice, static_cast<long long>(n_total), lr * grad_scale,
                                 init_master, static_cast<cudaStream_t>(stream)));
    return PW_OK;
}

// Device buffers that other processes can map.  Allocated here with cudaMalloc (a whole allocation
// of its own: the handle then names exactly this buffer) and opened by the other replicas with
// lazy peer access, which covers both another process on the same GPU and a process on a peer GPU.
namespace {
std::mutex g_shared_mu;
std::map<void*, int> g_shared_owned;     // pointers from pw_shared_alloc
std::map<void*, int> g_shared_opened;    // pointers from pw_shared_open
}  // namespace

pw_status_t pw_shared_alloc(size_t bytes, void** dev_ptr, pw_ipc_handle_t* handle)
{
    if (!dev_ptr || !handle || bytes == 0) return fail(PW_ERR_INVALID_ARG, "shared alloc: NULL output or zero size");
    static_assert(sizeof(cudaIpcMemHandle_t) <= sizeof(handle->bytes), "handle too small");
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) return fail_cuda("shared alloc", e);
    cudaIpcMemHandle_t h;
    e = cudaIpcGetMemHandle(&h, p);
    if (e != cudaSuccess) { cudaFree(p); return fail_cuda("shared alloc: export handle", e); }
    std::memset(handle->bytes, 0, sizeof(handle->bytes));
    std::memcpy(handle->bytes, &h, sizeof(h));
    { std::lock_guard<std::mutex> lock(g_shared_mu); g_shared_owned[p] = 1; }
    *dev_ptr = p;
    return PW_OK;
}

pw_status_t pw_shared_free(void* dev_ptr)
{
    {
        std::lock_guard<std::mutex> lock(g_shared_mu);
        auto it = g_shared_owned.find(dev_ptr);
        if (it == g_shared_owned.end()) return fail(PW_ERR_INVALID_ARG, "shared free: not a pointer from pw_shared_alloc");
        g_shared_owned.erase(it);
    }
    const cudaError_t e = cudaFree(dev_ptr);
    return e == cudaSuccess ? PW_OK : fail_cuda("shared free", e);
}

pw_status_t pw_shared_open(const pw_ipc_handle_t* handle, void** dev_ptr)
{
    if (!handle || !dev_ptr) return fail(PW_ERR_INVALID_ARG, "shared open: NULL argument");
    cudaIpcMemHandle_t h;
    std::memcpy(&h, handle->bytes, sizeof(h));
    void* p = nullptr;
    const cudaError_t e = cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess);
    if (e != cudaSuccess) return fail_cuda("shared open (a handle cannot be opened by the process that made it)", e);
    { std::lock_guard<std::mutex> lock(g_shared_mu); g_shared_opened[p] = 1; }
    *dev_ptr = p;
    return PW_OK;
}

pw_status_t pw_shared_close(void* dev_ptr)
{
    {
        std::lock_guard<std::mutex> lock(g_shared_mu);
        auto it = g_shared_opened.find(dev_ptr);
        if (it == g_shared_opened.end()) return fail(PW_ERR_INVALID_ARG, "shared close: not a pointer from pw_shared_open");
        g_shared_opened.erase(it);
    }
    const cudaError_t e = cudaIpcCloseMemHandle(dev_ptr);
    return e == cudaSuccess ? PW_OK : fail_cuda("shared close", e);
}

pw_status_t pw_op_selftest_wait_timeout(uint64_t limit_cycles, int* kernel_returned, void* stream)
{
    PW_RT_OR_FAIL();
    if (!kernel_returned) return fail(PW_ERR_INVALID_ARG, "kernel_returned is NULL");
    long long limit = static_cast<long long>(limit_cycles);
    if (limit < 1000) limit = 1000;
    if (limit > 2000000000ll) limit = 2000000000ll;            // about a second at most
    int* flag = nullptr;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&flag), sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(flag, 0, sizeof(int));
    if (e != cudaSuccess) { if (flag) cudaFree(flag); return fail_cuda("self-test flag", e); }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const char* err = launch_wait_selftest(rt->op_status, limit, flag, st);
    if (!err) {
        e = cudaStreamSynchronize(st);
        if (e == cudaSuccess) e = cudaMemcpy(kernel_returned, flag, sizeof(int), cudaMemcpyDeviceToHost);
    }
    cudaFree(flag);
    if (err) return fail(PW_ERR_CUDA, err);
    return e == cudaSuccess ? PW_OK : fail_cuda("self-test", e);
}

pw_status_t pw_set_log(int level, pw_log_fn fn, void* user)
{
    if (level < PW_LOG_OFF || level > PW_LOG_INFO) return fail(PW_ERR_INVALID_ARG, "unknown log level");
    std::lock_guard<std::mutex> lock(g_log_mu);
    g_log.level = level; g_log.fn = fn; g_log.user = user;
    return PW_OK;
}

pw_status_t pw_set_tuning(int knob, int value)
{
    Tuning& t = tuning();
    switch (knob) {
        case PW_TUNE_PDL: if (value != 0 && value != 1) break; t.pdl = value; ++t.epoch; return PW_OK;
        case PW_TUNE_GEMM_PAIR: if (value != 0 && value != 1) break; t.gemm_pair = value; ++t.epoch; return PW_OK;
        case PW_TUNE_GEMM_BN: if (value != 0 && value != 128 && value != 192 && value != 256) break; t.gemm_bn = value; ++t.epoch; return PW_OK;
        case PW_TUNE_GEMM_SPLIT: if (value != 0 && value != 1) break; t.gemm_split = value; ++t.epoch; return PW_OK;
        case PW_TUNE_GEMM_SPLIT_MIN_K: if (value < 1) break; t.gemm_split_min_k = value; ++t.epoch; return PW_OK;
        case PW_TUNE_FAIL_LAUNCH: if (value < 0) break; t.fail_launch_countdown = value; return PW_OK;
        case PW_TUNE_NVTX: if (value != 0 && value != 1) break; t.nvtx = value; return PW_OK;
        default: return fail(PW_ERR_INVALID_ARG, "unknown tuning knob");
    }
    return fail(PW_ERR_INVALID_ARG, "value out of range for this tuning knob");
}

pw_status_t pw_get_tuning(int knob, int* value)
{
    if (!value) return fail(PW_ERR_INVALID_ARG, "value is NULL");
    const Tuning& t = tuning();
    switch (knob) {
        case PW_TUNE_PDL: *value = t.pdl; return PW_OK;
        case PW_TUNE_GEMM_PAIR: *value = t.gemm_pair; return PW_OK;
        case PW_TUNE_GEMM_BN: *value = t.gemm_bn; return PW_OK;
        case PW_TUNE_GEMM_SPLIT: *value = t.gemm_split; return PW_OK;
        case PW_TUNE_GEMM_SPLIT_MIN_K: *value = t.gemm_split_min_k; return PW_OK;
        case PW_TUNE_FAIL_LAUNCH: *value = t.fail_launch_countdown; return PW_OK;
        case PW_TUNE_NVTX: *value = t.nvtx; return PW_OK;
        default: return fail(PW_ERR_INVALID_ARG, "unknown tuning knob");
    }
}

pw_status_t pw_op_status_reset(void)
{
    PW_RT_OR_FAIL();
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemset(rt->op_status, 0, sizeof(DeviceStatus));   // the device is idle: code, site, counters, tickets
    return e == cudaSuccess ? PW_OK : fail_cuda("status reset", e);
}

pw_status_t pw_op_status(int* device_status, int* site)
{
    PW_RT_OR_FAIL();
    return read_status(rt->op_status, device_status, site);
}

}  // extern "C"
