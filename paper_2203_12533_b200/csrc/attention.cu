// Attention backward, host side: delta = rowsum(dO * O) (HBM-bound, below; skipped when the GEMM that
// produced dO already took the sums in its epilogue), then the two tcgen05 kernels of
// attention_bwd_sm100.cu (dq; dk and dv).
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
// The kernel is bound by instruction issue as much as by memory: 32-bit index arithmetic and
// two-wide fp32 multiply-adds.
__global__ void __launch_bounds__(256)
attn_delta_kernel(const __nv_bfloat16* o, const __nv_bfloat16* dout,
                  float* delta, int B, int S, int H, int dh)
{
    const unsigned per_head = dh / 8;                        // threads per (token, head): 8 or 16
    const unsigned total = static_cast<unsigned>(B) * S * H * per_head;
    const unsigned base = blockIdx.x * 1024u + threadIdx.x;
    grid_dep_launch();
    grid_dep_wait();
    uint4 a[4], g[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const unsigned idx = base + u * 256;
        a[u] = idx < total ? *reinterpret_cast<const uint4*>(o + static_cast<size_t>(idx) * 8) : make_uint4(0, 0, 0, 0);
        g[u] = idx < total ? *reinterpret_cast<const uint4*>(dout + static_cast<size_t>(idx) * 8) : make_uint4(0, 0, 0, 0);
    }
    float s[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        uint64_t acc = ffma2(pack_f32x2(bf16_lo(a[u].x), bf16_hi(a[u].x)), pack_f32x2(bf16_lo(g[u].x), bf16_hi(g[u].x)), 0ull);
        acc = ffma2(pack_f32x2(bf16_lo(a[u].y), bf16_hi(a[u].y)), pack_f32x2(bf16_lo(g[u].y), bf16_hi(g[u].y)), acc);
        acc = ffma2(pack_f32x2(bf16_lo(a[u].z), bf16_hi(a[u].z)), pack_f32x2(bf16_lo(g[u].z), bf16_hi(g[u].z)), acc);
        acc = ffma2(pack_f32x2(bf16_lo(a[u].w), bf16_hi(a[u].w)), pack_f32x2(bf16_lo(g[u].w), bf16_hi(g[u].w)), acc);
        float lo, hi;
        unpack_f32x2(acc, lo, hi);
        s[u] = lo + hi;
    }
    for (unsigned off = per_head >> 1; off > 0; off >>= 1) {
#pragma unroll
        for (int u = 0; u < 4; ++u) s[u] += __shfl_xor_sync(0xffffffffu, s[u], off);
    }
    if ((threadIdx.x & (per_head - 1)) == 0) {               // 1024 and 256 are multiples of per_head
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned idx = base + u * 256;
            if (idx < total) {
                const unsigned th = idx / per_head;          // token * H + head
                const unsigned t = th / H, h = th - t * H;
                const unsigned bb = t / S, sq = t - bb * S;
                delta[(static_cast<size_t>(bb) * H + h) * S + sq] = s[u];
            }
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
    if (o != nullptr) {                                      // o == nullptr: delta already holds rowsum(dout * o)
        const size_t total = static_cast<size_t>(B) * S * H * (dh / 8);
        if (total >= (1ull << 31)) return "attention: too many (token, head) pairs for the row-dot kernel";
        if (launch_k(attn_delta_kernel, dim3(static_cast<unsigned>((total + 1023) / 1024)), dim3(256), 0, stream,
                     static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(dout), static_cast<float*>(delta), B, S, H, dh) != cudaSuccess)
            return "attention delta launch failed";
    }
    if (const char* e = launch_attention_bwd_dq(rt, qkv, dout, lse, delta, B, S, H, dh, dqkv, status, stream)) return e;
    return launch_attention_bwd_dkdv(rt, qkv, dout, lse, delta, B, S, H, dh, dqkv, status, stream);
}

}  // namespace pw
