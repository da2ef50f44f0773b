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

}  // namespace

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
