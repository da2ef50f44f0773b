// Gradient apply.  In the paper's appendix trace of data-parallel training each island applies
// the gradients it received before the next step starts; the paper names no optimizer, so this
// is plain stochastic gradient descent on an fp32 master copy, with the bf16 working copy that
// the layer kernels read re-derived from it in the same pass:
//     master <- master - step * grad          (step = lr * grad_scale, one fused multiply-add)
//     param  =  bf16(master)                  (round to nearest even)
// Memory bound: 4 (grad) + 4 + 4 (master in and out) + 2 (param) = 14 bytes per element.  One
// launch serves up to kApplyMaxItems tensors: a CTA owns one chunk of kApplyChunk consecutive
// elements of one tensor and finds it from a prefix table in the kernel's parameter space, so a
// layer's twelve tensors (eight of them a few KB) cost one launch, not twelve.
#include "pw_kernels.h"

namespace pw {
namespace {

constexpr int kApplyThreads = 256;
constexpr int kApplyIters = 4;                                   // 8 elements per thread and iteration
constexpr int kApplyChunk = kApplyThreads * 8 * kApplyIters;     // elements per CTA

struct ApplyTable {
    __nv_bfloat16* param[kApplyMaxItems];
    float* master[kApplyMaxItems];
    const float* grad[kApplyMaxItems];
    long long n[kApplyMaxItems];
    int first_block[kApplyMaxItems + 1];                         // CTA range of item i: [first_block[i], first_block[i+1])
    int count;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <bool INIT>
__global__ void __launch_bounds__(kApplyThreads)
sgd_apply_kernel(const __grid_constant__ ApplyTable tab, float step)
{
    grid_dep_launch();
    int it = 0;
    while (it + 1 < tab.count && static_cast<int>(blockIdx.x) >= tab.first_block[it + 1]) ++it;
    __nv_bfloat16* param = tab.param[it];
    float* master = tab.master[it];
    const float* grad = tab.grad[it];
    const long long n = tab.n[it];
    const long long base = static_cast<long long>(static_cast<int>(blockIdx.x) - tab.first_block[it]) * kApplyChunk;
    const bool vec = ((reinterpret_cast<uintptr_t>(param) | reinterpret_cast<uintptr_t>(master) |
                       reinterpret_cast<uintptr_t>(grad)) & 15) == 0;
    grid_dep_wait();

    if (vec && base + kApplyChunk <= n) {
        // Full, aligned chunk: every load of the chunk is in flight before the first use.
        float4 g[kApplyIters][2], m[kApplyIters][2];
        uint4 pw_[kApplyIters];
#pragma unroll
        for (int j = 0; j < kApplyIters; ++j) {
            const long long i = base + (static_cast<long long>(j) * kApplyThreads + threadIdx.x) * 8;
            g[j][0] = __ldcs(reinterpret_cast<const float4*>(grad + i));
            g[j][1] = __ldcs(reinterpret_cast<const float4*>(grad + i) + 1);
            if (INIT) {
                pw_[j] = *reinterpret_cast<const uint4*>(param + i);
            } else {
                m[j][0] = __ldcs(reinterpret_cast<const float4*>(master + i));
                m[j][1] = __ldcs(reinterpret_cast<const float4*>(master + i) + 1);
            }
        }
#pragma unroll
        for (int j = 0; j < kApplyIters; ++j) {
            const long long i = base + (static_cast<long long>(j) * kApplyThreads + threadIdx.x) * 8;
            if (INIT) {
                const uint32_t w[4] = {pw_[j].x, pw_[j].y, pw_[j].z, pw_[j].w};
                float f[8];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    f[2 * q] = __uint_as_float(w[q] << 16);
                    f[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
                }
                m[j][0] = make_float4(f[0], f[1], f[2], f[3]);
                m[j][1] = make_float4(f[4], f[5], f[6], f[7]);
            }
            float4 a = m[j][0], b = m[j][1];
            a.x = fmaf(-step, g[j][0].x, a.x); a.y = fmaf(-step, g[j][0].y, a.y);
            a.z = fmaf(-step, g[j][0].z, a.z); a.w = fmaf(-step, g[j][0].w, a.w);
            b.x = fmaf(-step, g[j][1].x, b.x); b.y = fmaf(-step, g[j][1].y, b.y);
            b.z = fmaf(-step, g[j][1].z, b.z); b.w = fmaf(-step, g[j][1].w, b.w);
            __stcs(reinterpret_cast<float4*>(master + i), a);
            __stcs(reinterpret_cast<float4*>(master + i) + 1, b);
            uint4 o;
            o.x = pack_bf16x2(a.x, a.y); o.y = pack_bf16x2(a.z, a.w);
            o.z = pack_bf16x2(b.x, b.y); o.w = pack_bf16x2(b.z, b.w);
            *reinterpret_cast<uint4*>(param + i) = o;
        }
        return;
    }
    // Ragged tail of a tensor, or pointers that are not 16-byte aligned: one element at a time.
    const long long end = (base + kApplyChunk < n) ? base + kApplyChunk : n;
    for (long long i = base + threadIdx.x; i < end; i += kApplyThreads) {
        const float m0 = INIT ? __bfloat162float(param[i]) : master[i];
        const float m1 = fmaf(-step, grad[i], m0);
        master[i] = m1;
        param[i] = __float2bfloat16_rn(m1);
    }
}

// Data-parallel form over peer memory.  Every replica (one process per GPU) has the gradients and
// the bf16 parameters of all tensors in one flat buffer each, mapped into every other replica's
// address space.  Replica `rank` owns the elements [lo, hi) of the flat index space and keeps the
// fp32 master of that slice only.  For its slice this kernel
//     reads the gradient of every replica (plain loads from peer memory, rank order 0..world-1:
//     the sum has one fixed order), applies the step to its master slice, and
//     stores the new bf16 values into every replica's parameter buffer (plain stores to peers),
// i.e. reduce-scatter, optimizer step and all-gather of the working copy in one pass: 4 bytes per
// element come in over the links and 2 go out, instead of the 8 + 8 of an fp32 all-reduce followed
// by a local apply.  The kernel waits on nothing: the caller orders it after every replica's
// backward pass and orders the next forward pass after every replica's kernel (stream-ordered or
// host barriers), so a missing peer can delay the host but never spin a GPU.
struct DpTable {
    const float* grad[kDpMaxWorld];
    __nv_bfloat16* param[kDpMaxWorld];
};

__device__ __forceinline__ void add8(float (&acc)[8], const float4& a, const float4& b)
{
    acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
    acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
}

template <bool INIT>
__global__ void __launch_bounds__(kApplyThreads)
dp_reduce_apply_kernel(const __grid_constant__ DpTable tab, int world, int rank, float* master, long long lo,
                       long long hi, float step, int vec)
{
    grid_dep_launch();
    const long long i = lo + (static_cast<long long>(blockIdx.x) * kApplyThreads + threadIdx.x) * 8;
    grid_dep_wait();
    if (i >= hi) return;
    if (vec && i + 8 <= hi) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int k0 = 0; k0 < world; k0 += 4) {                       // four replicas' loads in flight at a time
            float4 g[4][2];
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (k0 + q < world) {
                    const float4* src = reinterpret_cast<const float4*>(tab.grad[k0 + q] + i);
                    g[q][0] = __ldcv(src);                             // peers rewrite these every step: never from L1
                    g[q][1] = __ldcv(src + 1);
                }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (k0 + q < world) add8(acc, g[q][0], g[q][1]);
        }
        float m[8];
        if (INIT) {
            const uint4 w = *reinterpret_cast<const uint4*>(tab.param[rank] + i);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                m[2 * q] = __uint_as_float(ww[q] << 16);
                m[2 * q + 1] = __uint_as_float(ww[q] & 0xffff0000u);
            }
        } else {
            const float4 a = __ldcs(reinterpret_cast<const float4*>(master + (i - lo)));
            const float4 b = __ldcs(reinterpret_cast<const float4*>(master + (i - lo)) + 1);
            m[0] = a.x; m[1] = a.y; m[2] = a.z; m[3] = a.w; m[4] = b.x; m[5] = b.y; m[6] = b.z; m[7] = b.w;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) m[e] = fmaf(-step, acc[e], m[e]);
        __stcs(reinterpret_cast<float4*>(master + (i - lo)), make_float4(m[0], m[1], m[2], m[3]));
        __stcs(reinterpret_cast<float4*>(master + (i - lo)) + 1, make_float4(m[4], m[5], m[6], m[7]));
        uint4 o;
        o.x = pack_bf16x2(m[0], m[1]); o.y = pack_bf16x2(m[2], m[3]);
        o.z = pack_bf16x2(m[4], m[5]); o.w = pack_bf16x2(m[6], m[7]);
        for (int k = 0; k < world; ++k) *reinterpret_cast<uint4*>(tab.param[k] + i) = o;
        return;
    }
    const long long end = (i + 8 < hi) ? i + 8 : hi;
    for (long long j = i; j < end; ++j) {
        float g = 0.f;
        for (int k = 0; k < world; ++k) g += *reinterpret_cast<const volatile float*>(tab.grad[k] + j);
        const float m0 = INIT ? __bfloat162float(tab.param[rank][j]) : master[j - lo];
        const float m1 = fmaf(-step, g, m0);
        master[j - lo] = m1;
        const __nv_bfloat16 w = __float2bfloat16_rn(m1);
        for (int k = 0; k < world; ++k) tab.param[k][j] = w;
    }
}

}  // namespace

void dp_slice(long long n_total, int world, int rank, long long* lo, long long* hi)
{
    long long per = (n_total + world - 1) / world;
    per = (per + 7) / 8 * 8;                                          // slices start on 16-byte boundaries of the bf16 buffer
    long long a = per * rank, b = a + per;
    if (a > n_total) a = n_total;
    if (b > n_total) b = n_total;
    *lo = a; *hi = b;
}

const char* launch_dp_reduce_apply(int rank, int world, const void* const* grads, void* const* params, void* master,
                                   long long n_total, float step, int init_master, cudaStream_t stream)
{
    if (world < 1 || world > kDpMaxWorld || rank < 0 || rank >= world) return "data-parallel apply: bad rank or world size";
    DpTable tab;
    uintptr_t bits = reinterpret_cast<uintptr_t>(master);
    for (int k = 0; k < kDpMaxWorld; ++k) {
        tab.grad[k] = k < world ? static_cast<const float*>(grads[k]) : nullptr;
        tab.param[k] = k < world ? static_cast<__nv_bfloat16*>(params[k]) : nullptr;
        if (k < world) bits |= reinterpret_cast<uintptr_t>(grads[k]) | reinterpret_cast<uintptr_t>(params[k]);
    }
    long long lo, hi;
    dp_slice(n_total, world, rank, &lo, &hi);
    if (hi <= lo) return nullptr;                                     // this replica owns nothing
    const long long per_block = static_cast<long long>(kApplyThreads) * 8;
    const long long blocks = (hi - lo + per_block - 1) / per_block;
    if (blocks > 0x7fffffffll) return "data-parallel apply: too many elements for one call";
    const int vec = (bits & 15) == 0;
    const cudaError_t e = init_master
        ? launch_k(dp_reduce_apply_kernel<true>, dim3(static_cast<unsigned>(blocks)), dim3(kApplyThreads), 0, stream, tab, world, rank,
                   static_cast<float*>(master), lo, hi, step, vec)
        : launch_k(dp_reduce_apply_kernel<false>, dim3(static_cast<unsigned>(blocks)), dim3(kApplyThreads), 0, stream, tab, world, rank,
                   static_cast<float*>(master), lo, hi, step, vec);
    return e == cudaSuccess ? nullptr : "data-parallel apply launch failed";
}

const char* launch_sgd_apply(const ApplyItem* items, int n_items, float step, int init_master, cudaStream_t stream)
{
    int done = 0;
    while (done < n_items) {
        ApplyTable tab;
        int count = 0;
        long long blocks = 0;
        while (done < n_items && count < kApplyMaxItems) {
            const ApplyItem& a = items[done++];
            if (a.n == 0) continue;
            tab.param[count] = static_cast<__nv_bfloat16*>(a.param);
            tab.master[count] = static_cast<float*>(a.master);
            tab.grad[count] = static_cast<const float*>(a.grad);
            tab.n[count] = a.n;
            tab.first_block[count] = static_cast<int>(blocks);
            blocks += (a.n + kApplyChunk - 1) / kApplyChunk;
            if (blocks > 0x7fffffffll) return "gradient apply: too many elements for one call";
            ++count;
        }
        if (count == 0) continue;
        for (int i = count; i <= kApplyMaxItems; ++i) tab.first_block[i] = static_cast<int>(blocks);
        for (int i = count; i < kApplyMaxItems; ++i) {
            tab.param[i] = nullptr; tab.master[i] = nullptr; tab.grad[i] = nullptr; tab.n[i] = 0;
        }
        tab.count = count;
        const cudaError_t e = init_master
            ? launch_k(sgd_apply_kernel<true>, dim3(static_cast<unsigned>(blocks)), dim3(kApplyThreads), 0, stream, tab, step)
            : launch_k(sgd_apply_kernel<false>, dim3(static_cast<unsigned>(blocks)), dim3(kApplyThreads), 0, stream, tab, step);
        if (e != cudaSuccess) return "gradient apply launch failed";
    }
    return nullptr;
}

}  // namespace pw
