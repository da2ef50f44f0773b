// First and last layer of the decoder language model (Section 5.3: "an embedding layer first and a
// softmax layer last"): embedding lookup and its deterministic scatter-add backward, and the fused
// softmax / cross-entropy over the logits of the tied output projection (the projection itself and
// its two backward products are the tcgen05 GEMMs of gemm_sm100.cu).  All HBM-bound: 16-byte
// accesses, fp32 arithmetic, fixed-order reductions (bitwise reproducible).
#include "pw_kernels.h"

namespace pw {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kStatusBadIndex = 1;   // == PW_ERR_INVALID_ARG: a token id or label outside [0, V)

// ------------------------------------------------------------------------------------ embedding lookup
// x0[t][:] = E[ids[t]][:].  One 16-byte piece per thread; an id outside [0, V) is recorded in the
// status word and reads row 0.
__global__ void __launch_bounds__(256)
embed_gather_kernel(const int* ids, const __nv_bfloat16* E, int T, int d, int V, __nv_bfloat16* x0, DeviceStatus* status)
{
    grid_dep_launch();
    grid_dep_wait();
    const int per_row = d / 8;
    const size_t total = static_cast<size_t>(T) * per_row;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const int t = static_cast<int>(i / per_row), c = static_cast<int>(i % per_row);
        int id = ids[t];
        if (id < 0 || id >= V) {
            if (c == 0) atomicCAS(&status->code, 0, kStatusBadIndex);
            id = 0;
        }
        reinterpret_cast<uint4*>(x0)[i] = *reinterpret_cast<const uint4*>(E + static_cast<size_t>(id) * d + c * 8);
    }
}

// ------------------------------------------------------------------------------------ embedding backward
// dE[v][:] += sum over the tokens t with ids[t] == v of dx0[t][:], tokens added in increasing t, so
// the result does not depend on scheduling.  Step 1 threads every token onto a per-row list
// (head[v], next[t]; the order of a list depends on timing, its content does not); step 2 gives a
// warp to every vocabulary row: the warp ranks the row's tokens (all-pairs compare for up to 32,
// repeated minimum search beyond) and adds their rows in rank order.
__global__ void __launch_bounds__(256)
embed_link_kernel(const int* ids, int T, int V, int* head, int* next, DeviceStatus* status)
{
    grid_dep_launch();
    grid_dep_wait();
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const int id = ids[t];
    if (id < 0 || id >= V) { atomicCAS(&status->code, 0, kStatusBadIndex); next[t] = -1; return; }
    next[t] = atomicExch(&head[id], t);
}

__global__ void __launch_bounds__(256)
embed_scatter_kernel(const __nv_bfloat16* dx0, int d, int V, const int* head, const int* next, float* dE)
{
    grid_dep_launch();
    grid_dep_wait();
    const int v = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (v >= V) return;
    const int first = head[v];
    if (first < 0) return;
    int n = 0, mine = -1;
    for (int t = first; t >= 0; t = next[t], ++n)
        if (n == lane) mine = t;                            // lane i keeps the i-th list entry (first 32 entries)
    float* out = dE + static_cast<size_t>(v) * d;
    auto add_row = [&](int t) {
        const __nv_bfloat16* src = dx0 + static_cast<size_t>(t) * d;
        for (int c = lane * 8; c < d; c += 256) {
            float f[8];
            unpack8(*reinterpret_cast<const uint4*>(src + c), f);
            float4 a = *reinterpret_cast<float4*>(out + c), b = *reinterpret_cast<float4*>(out + c + 4);
            a.x += f[0]; a.y += f[1]; a.z += f[2]; a.w += f[3];
            b.x += f[4]; b.y += f[5]; b.z += f[6]; b.w += f[7];
            *reinterpret_cast<float4*>(out + c) = a;
            *reinterpret_cast<float4*>(out + c + 4) = b;
        }
    };
    if (n <= 32) {
        // rank = number of entries with a smaller token index
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const int other = __shfl_sync(0xffffffffu, mine, j);
            rank += (lane < n && other < mine) ? 1 : 0;
        }
        for (int r = 0; r < n; ++r) {
            const unsigned who = __ballot_sync(0xffffffffu, lane < n && rank == r);
            const int t = __shfl_sync(0xffffffffu, mine, __ffs(who) - 1);
            add_row(t);
        }
    } else {
        int last = -1;
        for (int r = 0; r < n; ++r) {                       // next smallest index above `last`
            int best = 0x7fffffff;
            for (int t = first; t >= 0; t = next[t])
                if (t > last && t < best) best = t;
            add_row(best);
            last = best;
        }
    }
}

// ------------------------------------------------------------------------------------ softmax / cross-entropy
// One CTA per token row of the logits z (bf16 [T, ld], V columns used):
//   lse = log sum_v exp z_v   (one pass with a running maximum per thread, then a fixed-order
//                              combination across the CTA)
//   loss_row = lse - z[label]
//   z_v <- grad_scale * (exp(z_v - lse) - [v == label])      written back in place as bf16
// The row (64 KB at V = 32768) is read twice; the second read comes from L2.
constexpr int kXentThreads = 256;

__global__ void __launch_bounds__(kXentThreads)
softmax_xent_kernel(__nv_bfloat16* logits, int ld, const int* labels, int V, float grad_scale, float* lse_out,
                    float* loss_rows, DeviceStatus* status)
{
    __shared__ float red_m[kXentThreads / 32], red_s[kXentThreads / 32];
    __shared__ float sh_lse;
    grid_dep_launch();
    grid_dep_wait();
    const int t = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __nv_bfloat16* row = logits + static_cast<size_t>(t) * ld;
    float m = -INFINITY, s = 0.f;                           // running maximum (log2 units) and sum of 2^(z' - m)
    for (int c = threadIdx.x * 8; c < V; c += kXentThreads * 8) {
        float f[8];
        unpack8(*reinterpret_cast<const uint4*>(row + c), f);
        float mx = f[0];
#pragma unroll
        for (int k = 1; k < 8; ++k) mx = fmaxf(mx, f[k]);
        mx *= kLog2e;
        if (mx > m) { s *= ex2_approx(m - mx); m = mx; }
#pragma unroll
        for (int k = 0; k < 8; ++k) s += ex2_approx(fmaf(f[k], kLog2e, -m));
    }
    // combine (m, s) pairs: lanes by shuffles, warps in order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
        const float mn = fmaxf(m, m2);
        s = (m == -INFINITY ? 0.f : s * ex2_approx(m - mn)) + (m2 == -INFINITY ? 0.f : s2 * ex2_approx(m2 - mn));
        m = mn;
    }
    if (lane == 0) { red_m[warp] = m; red_s[warp] = s; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float mm = red_m[0], ss = red_s[0];
        for (int w = 1; w < kXentThreads / 32; ++w) {
            const float mn = fmaxf(mm, red_m[w]);
            ss = (mm == -INFINITY ? 0.f : ss * ex2_approx(mm - mn)) + (red_m[w] == -INFINITY ? 0.f : red_s[w] * ex2_approx(red_m[w] - mn));
            mm = mn;
        }
        const float lse = (mm + log2f(ss)) * kLn2;
        int label = labels[t];
        if (label < 0 || label >= V) { atomicCAS(&status->code, 0, kStatusBadIndex); label = 0; }
        sh_lse = lse;
        lse_out[t] = lse;
        loss_rows[t] = lse - __bfloat162float(row[label]);
    }
    __syncthreads();
    const float nl2 = -sh_lse * kLog2e;
    int label = labels[t];
    if (label < 0 || label >= V) label = 0;
    for (int c = threadIdx.x * 8; c < V; c += kXentThreads * 8) {
        float f[8];
        unpack8(*reinterpret_cast<const uint4*>(row + c), f);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float g = ex2_approx(fmaf(f[k], kLog2e, nl2));
            if (c + k == label) g -= 1.0f;
            f[k] = g * grad_scale;
        }
        *reinterpret_cast<uint4*>(row + c) = pack8(f);
    }
}

// out[0] = scale * sum of in[0..n), summed in a fixed order (thread i adds elements i, i+1024, ...;
// then a fixed tree).
__global__ void __launch_bounds__(1024)
sum_scale_kernel(const float* in, int n, float scale, float* out)
{
    __shared__ float red[1024];
    grid_dep_launch();
    grid_dep_wait();
    float s = 0.f;
    for (int i = threadIdx.x; i < n; i += 1024) s += in[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) out[0] = red[0] * scale;
}

}  // namespace

const char* launch_embedding_fwd(Runtime* rt, const void* ids, const void* E, int T, int d, int V, void* x0,
                                 DeviceStatus* status, cudaStream_t stream)
{
    if (T <= 0 || V <= 0 || d <= 0 || (d % 8)) return "embedding: d must be a positive multiple of 8";
    const size_t total = static_cast<size_t>(T) * (d / 8);
    size_t blocks = (total + 255) / 256;
    const size_t cap = static_cast<size_t>(rt->sm_count) * 16;
    if (blocks > cap) blocks = cap;
    return launch_k(embed_gather_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream,
                    static_cast<const int*>(ids), static_cast<const __nv_bfloat16*>(E), T, d, V,
                    static_cast<__nv_bfloat16*>(x0), status) == cudaSuccess
               ? nullptr : "embedding lookup launch failed";
}

size_t embedding_bwd_scratch_bytes(int T, int V)
{
    if (T <= 0 || V <= 0) return 0;
    return (static_cast<size_t>(T) + static_cast<size_t>(V)) * sizeof(int);
}

const char* launch_embedding_bwd(Runtime* rt, const void* ids, const void* dx0, int T, int d, int V, void* dE,
                                 void* scratch, DeviceStatus* status, cudaStream_t stream)
{
    (void)rt;
    if (T <= 0 || V <= 0 || d <= 0 || (d % 8)) return "embedding: d must be a positive multiple of 8";
    int* head = static_cast<int*>(scratch);
    int* next = head + V;
    if (cudaMemsetAsync(head, 0xff, static_cast<size_t>(V) * sizeof(int), stream) != cudaSuccess) return "embedding bwd: memset failed";
    if (launch_k(embed_link_kernel, dim3((T + 255) / 256), dim3(256), 0, stream, static_cast<const int*>(ids), T, V, head,
                 next, status) != cudaSuccess)
        return "embedding bwd (link) launch failed";
    return launch_k(embed_scatter_kernel, dim3((V + 7) / 8), dim3(256), 0, stream, static_cast<const __nv_bfloat16*>(dx0), d, V,
                    static_cast<const int*>(head), static_cast<const int*>(next), static_cast<float*>(dE)) == cudaSuccess
               ? nullptr : "embedding bwd (scatter) launch failed";
}

const char* launch_softmax_xent(Runtime* rt, void* logits, int ld, const void* labels, int T, int V, float grad_scale,
                                void* lse, void* loss_rows, DeviceStatus* status, cudaStream_t stream)
{
    (void)rt;
    if (T <= 0 || V <= 0 || (V % 8) || (ld % 8) || ld < V) return "softmax-xent: V and ld must be multiples of 8, ld >= V";
    return launch_k(softmax_xent_kernel, dim3(T), dim3(kXentThreads), 0, stream, static_cast<__nv_bfloat16*>(logits), ld,
                    static_cast<const int*>(labels), V, grad_scale, static_cast<float*>(lse), static_cast<float*>(loss_rows),
                    status) == cudaSuccess
               ? nullptr : "softmax-xent launch failed";
}

const char* launch_sum_scale(const void* in, int n, float scale, void* out, cudaStream_t stream)
{
    if (n <= 0) return "sum: empty input";
    return launch_k(sum_scale_kernel, dim3(1), dim3(1024), 0, stream, static_cast<const float*>(in), n, scale,
                    static_cast<float*>(out)) == cudaSuccess
               ? nullptr : "sum launch failed";
}

}  // namespace pw
