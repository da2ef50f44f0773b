// Attention backward, host side: delta = rowsum(dO * O) (HBM-bound, below), then the two tcgen05
// kernels of attention_bwd_sm100.cu (dq; dk and dv).
#include "pw_kernels.h"

namespace pw {

const char* launch_attention_bwd_dq(Runtime* rt, const void* qkv, const void* dout, const void* lse, const void* delta,
                                    int B, int S, int H, int dh, void* dqkv, DeviceStatus* status, cudaStream_t stream);
const char* launch_attention_bwd_dkdv(Runtime* rt, const void* qkv, const void* dout, const void* lse, const void* delta,
                                      int B, int S, int H, int dh, void* dqkv, DeviceStatus* status, cudaStream_t stream);
const char* configure_attention_bwd_tc();

namespace {

// ------------------------------------------------------------------------------------ delta = rowsum(dout * o)
// Each thread handles four 16-byte pieces that are a whole block stride apart (all eight loads
// are issued before any is used); the dh/8 threads of a (token, head) group reduce by shuffles.
__global__ void __launch_bounds__(256)
attn_delta_kernel(const __nv_bfloat16* o, const __nv_bfloat16* dout,
                  float* delta, int B, int S, int H, int dh)
{
    const int per_head = dh / 8;                             // threads per (token, head): 8 or 16
    const size_t total = static_cast<size_t>(B) * S * H * per_head;
    const size_t base = static_cast<size_t>(blockIdx.x) * 1024 + threadIdx.x;
    grid_dep_launch();
    grid_dep_wait();
    uint4 a[4], g[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const size_t idx = base + u * 256;
        a[u] = idx < total ? *reinterpret_cast<const uint4*>(o + idx * 8) : make_uint4(0, 0, 0, 0);
        g[u] = idx < total ? *reinterpret_cast<const uint4*>(dout + idx * 8) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const size_t idx = base + u * 256;
        float fa[8], fg[8];
        unpack8(a[u], fa);
        unpack8(g[u], fg);
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) s += fa[k] * fg[k];
        for (int off = per_head >> 1; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (idx < total && (idx % per_head) == 0) {
            const size_t th = idx / per_head;                // token * H + head
            const size_t t = th / H, h = th % H;
            const size_t bb = t / S, sq = t % S;
            delta[(bb * H + h) * S + sq] = s;
        }
    }
}

}  // namespace

const char* configure_attention() { return configure_attention_bwd_tc(); }

const char* launch_attention_bwd(Runtime* rt, const void* qkv, const void* o, const void* dout, const void* lse,
                                 int B, int S, int H, int dh, void* dqkv, void* delta, DeviceStatus* status,
                                 cudaStream_t stream)
{
    if (B <= 0 || H <= 0 || S <= 0 || (S % 128) != 0 || (dh != 64 && dh != 128)) return "attention: unsupported shape";
    {
        const size_t total = static_cast<size_t>(B) * S * H * (dh / 8);
        if (launch_k(attn_delta_kernel, dim3(static_cast<unsigned>((total + 1023) / 1024)), dim3(256), 0, stream,
                     static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(dout), static_cast<float*>(delta), B, S, H, dh) != cudaSuccess)
            return "attention delta launch failed";
    }
    if (const char* e = launch_attention_bwd_dq(rt, qkv, dout, lse, delta, B, S, H, dh, dqkv, status, stream)) return e;
    return launch_attention_bwd_dkdv(rt, qkv, dout, lse, delta, B, S, H, dh, dqkv, status, stream);
}

}  // namespace pw
