// Causal attention backward (never materialises the S x S score matrix).  Warp-level
// tensor-core path (mma.sync m16n8k16 bf16, fp32 accumulate), cp.async double-buffered tiles in
// XOR-swizzled shared memory, ldmatrix operand fetch.  (The forward is in attention_fwd_sm100.cu.)
//
//   backward  : delta = rowsum(dout * o); then two kernels so that every output is owned by one
//               CTA (no atomics, bitwise reproducible):
//                 dq   : CTA = 128 queries, loops over key/value tiles (S, dP, then dQ += dS K)
//                 dkdv : CTA = 128 keys, loops over query tiles (S^T, dP^T, dV += P^T dO, dK += dS^T Q)
//
// Packed layout: qkv[T, 3d], q at column h*dh, k at d + h*dh, v at 2d + h*dh; o/dout [T, d].
#include "pw_kernels.h"

namespace pw {
namespace {

constexpr int kAttnThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A [rows][DH] bf16 tile in shared memory; the 16-byte chunk c of row r lives at chunk c ^ (r & 7).
template <int DH>
struct Tile {
    static constexpr int kRowBytes = DH * 2;
    static constexpr int kChunks = DH / 8;
    __device__ static uint32_t addr(uint32_t base, int r, int c /*multiple of 8*/)
    {
        return base + r * kRowBytes + ((((c >> 3) ^ (r & 7))) << 4);
    }
    // Cooperative async copy of `rows` rows starting at global row pointer g (row pitch ld elements).
    __device__ static void load(uint32_t base, const __nv_bfloat16* g, int ld, int rows)
    {
        for (int i = threadIdx.x; i < rows * kChunks; i += kAttnThreads) {
            const int r = i / kChunks, ch = i % kChunks;
            cp_async16(base + r * kRowBytes + ((ch ^ (r & 7)) << 4), g + static_cast<size_t>(r) * ld + ch * 8);
        }
    }
};

// A-operand fragment (16 rows x 16 k) at rows r0.., columns c0.. of a row-major tile.
template <int DH>
__device__ __forceinline__ void load_a(uint32_t base, int r0, int c0, uint32_t* a)
{
    const int lane = threadIdx.x & 31;
    ldsm_x4(Tile<DH>::addr(base, r0 + (lane & 7) + ((lane >> 3) & 1) * 8, c0 + (lane >> 4) * 8), a[0], a[1], a[2], a[3]);
}
// B-operand fragments for two adjacent n-blocks (16 n) x 16 k, where the tile row is n and the
// tile column is k:  (b[0], b[1]) -> n-block n0, (b[2], b[3]) -> n-block n0 + 8.
template <int DH>
__device__ __forceinline__ void load_b_nk(uint32_t base, int n0, int k0, uint32_t* b)
{
    const int lane = threadIdx.x & 31;
    ldsm_x4(Tile<DH>::addr(base, n0 + (lane & 7) + (lane >> 4) * 8, k0 + ((lane >> 3) & 1) * 8), b[0], b[1], b[2], b[3]);
}
// Same, where the tile row is k and the tile column is n (transposing load).
template <int DH>
__device__ __forceinline__ void load_b_kn(uint32_t base, int k0, int n0, uint32_t* b)
{
    const int lane = threadIdx.x & 31;
    ldsm_x4_t(Tile<DH>::addr(base, k0 + (lane & 7) + ((lane >> 3) & 1) * 8, n0 + (lane >> 4) * 8), b[0], b[1], b[2], b[3]);
}

__device__ __forceinline__ float quad_max(float v)
{
    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
    return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v)
{
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

// Writes a warp's 16 x DH fp32 accumulator (scaled) as bf16 into its own 16 rows of a shared
// tile, then copies those rows to global memory with 16-byte stores.
template <int DH>
__device__ __forceinline__ void store_rows16(uint32_t tile_base, uint8_t* tile_ptr, int r0, const float (*acc)[4],
                                             float s_lo, float s_hi, __nv_bfloat16* g, int ld)
{
    const int lane = threadIdx.x & 31;
    __syncwarp();
#pragma unroll
    for (int nb = 0; nb < DH / 8; ++nb) {
        const int c = nb * 8 + 2 * (lane & 3);
        const int rl = r0 + (lane >> 2), rh = rl + 8;
        const uint32_t lo = pack_bf16(acc[nb][0] * s_lo, acc[nb][1] * s_lo);
        const uint32_t hi = pack_bf16(acc[nb][2] * s_hi, acc[nb][3] * s_hi);
        *reinterpret_cast<uint32_t*>(tile_ptr + (Tile<DH>::addr(tile_base, rl, c & ~7) - tile_base) + (c & 7) * 2) = lo;
        *reinterpret_cast<uint32_t*>(tile_ptr + (Tile<DH>::addr(tile_base, rh, c & ~7) - tile_base) + (c & 7) * 2) = hi;
    }
    __syncwarp();
    for (int i = lane; i < 16 * Tile<DH>::kChunks; i += 32) {
        const int r = r0 + i / Tile<DH>::kChunks, ch = i % Tile<DH>::kChunks;
        const uint4 v = *reinterpret_cast<const uint4*>(tile_ptr + (Tile<DH>::addr(tile_base, r, ch * 8) - tile_base));
        *reinterpret_cast<uint4*>(g + static_cast<size_t>(r - r0) * ld + ch * 8) = v;
    }
}

// ------------------------------------------------------------------------------------ delta = rowsum(dout * o)
__global__ void attn_delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ dout,
                                  float* __restrict__ delta, int B, int S, int H, int dh)
{
    const int per_head = dh / 8;                             // threads per (token, head): 8 or 16
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t total = static_cast<size_t>(B) * S * H * per_head;
    float s = 0.f;
    if (idx < total) {
        float a[8], g[8];
        unpack8(*reinterpret_cast<const uint4*>(o + idx * 8), a);
        unpack8(*reinterpret_cast<const uint4*>(dout + idx * 8), g);
#pragma unroll
        for (int k = 0; k < 8; ++k) s += a[k] * g[k];
    }
    for (int off = per_head >> 1; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (idx < total && (idx % per_head) == 0) {
        const size_t th = idx / per_head;                    // token * H + head
        const size_t t = th / H, h = th % H;
        const size_t b = t / S, sq = t % S;
        delta[(b * H + h) * S + sq] = s;
    }
}

// ------------------------------------------------------------------------------------ backward: dq
template <int DH>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_bwd_dq_kernel(const __nv_bfloat16* __restrict__ qkv, const __nv_bfloat16* __restrict__ dout,
                   const float* __restrict__ lse, const float* __restrict__ delta, __nv_bfloat16* __restrict__ dqkv,
                   int S, int H, float scale)
{
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int QB = 128 * DH * 2, KB = 64 * DH * 2;
    const uint32_t sQ = smem_u32(smem), sG = sQ + QB, sK = sG + QB, sV = sK + 2 * KB;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qblk = gridDim.x - 1 - blockIdx.x;
    const int b = blockIdx.y / H, h = blockIdx.y % H;
    const int d = H * DH, ld = 3 * d;
    const int q0 = qblk * 128;
    const __nv_bfloat16* gq = qkv + static_cast<size_t>(b * S + q0) * ld + h * DH;
    const __nv_bfloat16* gg = dout + static_cast<size_t>(b * S + q0) * d + h * DH;
    const __nv_bfloat16* gk = qkv + static_cast<size_t>(b * S) * ld + d + h * DH;
    const __nv_bfloat16* gv = gk + d;
    const int n_tiles = (q0 + 128) / 64;
    const float sl2 = scale * kLog2e;

    Tile<DH>::load(sQ, gq, ld, 128);
    Tile<DH>::load(sG, gg, d, 128);
    Tile<DH>::load(sK, gk, ld, 64);
    Tile<DH>::load(sV, gv, ld, 64);
    cp_async_commit();

    const int row_lo = q0 + warp * 16 + (lane >> 2), row_hi = row_lo + 8;
    const float* L = lse + (static_cast<size_t>(b) * H + h) * S;
    const float* Dl = delta + (static_cast<size_t>(b) * H + h) * S;
    const float lse_lo = L[row_lo] * kLog2e, lse_hi = L[row_hi] * kLog2e;
    const float dl_lo = Dl[row_lo], dl_hi = Dl[row_hi];
    float dq[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f;

    for (int t = 0; t < n_tiles; ++t) {
        const int buf = t & 1;
        if (t + 1 < n_tiles) {
            Tile<DH>::load(sK + (buf ^ 1) * KB, gk + static_cast<size_t>(t + 1) * 64 * ld, ld, 64);
            Tile<DH>::load(sV + (buf ^ 1) * KB, gv + static_cast<size_t>(t + 1) * 64 * ld, ld, 64);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const int kv0 = t * 64;
        if (kv0 <= q0 + warp * 16 + 15) {
            const uint32_t kb = sK + buf * KB, vb = sV + buf * KB;
            float sacc[8][4], pacc[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
                pacc[i][0] = pacc[i][1] = pacc[i][2] = pacc[i][3] = 0.f;
            }
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
                uint32_t qa[4], ga[4];
                load_a<DH>(sQ, warp * 16, ks * 16, qa);
                load_a<DH>(sG, warp * 16, ks * 16, ga);
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t bb[4];
                    load_b_nk<DH>(kb, np * 16, ks * 16, bb);
                    mma16816(sacc[2 * np], qa, bb[0], bb[1]);
                    mma16816(sacc[2 * np + 1], qa, bb[2], bb[3]);
                    load_b_nk<DH>(vb, np * 16, ks * 16, bb);
                    mma16816(pacc[2 * np], ga, bb[0], bb[1]);
                    mma16816(pacc[2 * np + 1], ga, bb[2], bb[3]);
                }
            }
            const bool diag = kv0 + 63 > q0 + warp * 16;
            uint32_t dsf[4][4];
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
                const int c = kv0 + nb * 8 + 2 * (lane & 3);
                float p0 = exp2f(sacc[nb][0] * sl2 - lse_lo), p1 = exp2f(sacc[nb][1] * sl2 - lse_lo);
                float p2 = exp2f(sacc[nb][2] * sl2 - lse_hi), p3 = exp2f(sacc[nb][3] * sl2 - lse_hi);
                if (diag) {
                    if (c > row_lo) p0 = 0.f;
                    if (c + 1 > row_lo) p1 = 0.f;
                    if (c > row_hi) p2 = 0.f;
                    if (c + 1 > row_hi) p3 = 0.f;
                }
                const float d0 = p0 * (pacc[nb][0] - dl_lo), d1 = p1 * (pacc[nb][1] - dl_lo);
                const float d2 = p2 * (pacc[nb][2] - dl_hi), d3 = p3 * (pacc[nb][3] - dl_hi);
                dsf[nb >> 1][(nb & 1) * 2] = pack_bf16(d0, d1);
                dsf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(d2, d3);
            }
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
                for (int np = 0; np < DH / 16; ++np) {
                    uint32_t bb[4];
                    load_b_kn<DH>(kb, ks * 16, np * 16, bb);
                    mma16816(dq[2 * np], dsf[ks], bb[0], bb[1]);
                    mma16816(dq[2 * np + 1], dsf[ks], bb[2], bb[3]);
                }
            }
        }
        __syncthreads();
    }
    store_rows16<DH>(sQ, smem, warp * 16, dq, scale, scale,
                     dqkv + static_cast<size_t>(b * S + q0 + warp * 16) * ld + h * DH, ld);
}

// ------------------------------------------------------------------------------------ backward: dk, dv
template <int DH>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_bwd_dkdv_kernel(const __nv_bfloat16* __restrict__ qkv, const __nv_bfloat16* __restrict__ dout,
                     const float* __restrict__ lse, const float* __restrict__ delta,
                     __nv_bfloat16* __restrict__ dqkv, int S, int H, float scale)
{
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int KBk = 128 * DH * 2, QB = 64 * DH * 2;
    const uint32_t sK = smem_u32(smem), sV = sK + KBk, sQ = sV + KBk, sG = sQ + 2 * QB;
    float* sL = reinterpret_cast<float*>(smem + 2 * KBk + 4 * QB);   // [2][64] lse * log2e
    float* sD = sL + 128;                                            // [2][64] delta
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kblk = blockIdx.x;                                     // key block 0 has the most query tiles
    const int b = blockIdx.y / H, h = blockIdx.y % H;
    const int d = H * DH, ld = 3 * d;
    const int k0 = kblk * 128;
    const __nv_bfloat16* gk = qkv + static_cast<size_t>(b * S + k0) * ld + d + h * DH;
    const __nv_bfloat16* gv = gk + d;
    const __nv_bfloat16* gq = qkv + static_cast<size_t>(b * S) * ld + h * DH;
    const __nv_bfloat16* gg = dout + static_cast<size_t>(b * S) * d + h * DH;
    const float* L = lse + (static_cast<size_t>(b) * H + h) * S;
    const float* Dl = delta + (static_cast<size_t>(b) * H + h) * S;
    const int t_begin = k0 / 64, t_end = S / 64;                     // query tiles that can see these keys
    const float sl2 = scale * kLog2e;

    auto load_q_tile = [&](int t, int buf) {
        Tile<DH>::load(sQ + buf * QB, gq + static_cast<size_t>(t) * 64 * ld, ld, 64);
        Tile<DH>::load(sG + buf * QB, gg + static_cast<size_t>(t) * 64 * d, d, 64);
        if (threadIdx.x < 64) {
            sL[buf * 64 + threadIdx.x] = L[t * 64 + threadIdx.x] * kLog2e;
            sD[buf * 64 + threadIdx.x] = Dl[t * 64 + threadIdx.x];
        }
    };
    Tile<DH>::load(sK, gk, ld, 128);
    Tile<DH>::load(sV, gv, ld, 128);
    load_q_tile(t_begin, 0);
    cp_async_commit();

    float dk[DH / 8][4], dv[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
        dk[i][0] = dk[i][1] = dk[i][2] = dk[i][3] = 0.f;
        dv[i][0] = dv[i][1] = dv[i][2] = dv[i][3] = 0.f;
    }
    const int key_lo = k0 + warp * 16 + (lane >> 2), key_hi = key_lo + 8;

    for (int t = t_begin; t < t_end; ++t) {
        const int buf = (t - t_begin) & 1;
        if (t + 1 < t_end) {
            load_q_tile(t + 1, buf ^ 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const int qt0 = t * 64;
        if (qt0 + 63 >= k0 + warp * 16) {                            // some query of the tile sees this warp's keys
            const uint32_t qb = sQ + buf * QB, gb = sG + buf * QB;
            const bool diag = qt0 < k0 + warp * 16 + 15;
#pragma unroll
            for (int half = 0; half < 2; ++half) {                   // 32 queries at a time keeps registers in check
                float sacc[4][4], pacc[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
                    pacc[i][0] = pacc[i][1] = pacc[i][2] = pacc[i][3] = 0.f;
                }
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    uint32_t ka[4], va[4];
                    load_a<DH>(sK, warp * 16, ks * 16, ka);
                    load_a<DH>(sV, warp * 16, ks * 16, va);
#pragma unroll
                    for (int np = 0; np < 2; ++np) {
                        uint32_t bb[4];
                        load_b_nk<DH>(qb, half * 32 + np * 16, ks * 16, bb);
                        mma16816(sacc[2 * np], ka, bb[0], bb[1]);
                        mma16816(sacc[2 * np + 1], ka, bb[2], bb[3]);
                        load_b_nk<DH>(gb, half * 32 + np * 16, ks * 16, bb);
                        mma16816(pacc[2 * np], va, bb[0], bb[1]);
                        mma16816(pacc[2 * np + 1], va, bb[2], bb[3]);
                    }
                }
                uint32_t pf[2][4], dsf[2][4];
#pragma unroll
                for (int nb = 0; nb < 4; ++nb) {
                    const int cl = half * 32 + nb * 8 + 2 * (lane & 3);   // query index inside the tile
                    const float l0 = sL[buf * 64 + cl], l1 = sL[buf * 64 + cl + 1];
                    const float e0 = sD[buf * 64 + cl], e1 = sD[buf * 64 + cl + 1];
                    float p0 = exp2f(sacc[nb][0] * sl2 - l0), p1 = exp2f(sacc[nb][1] * sl2 - l1);
                    float p2 = exp2f(sacc[nb][2] * sl2 - l0), p3 = exp2f(sacc[nb][3] * sl2 - l1);
                    if (diag) {
                        const int q = qt0 + cl;
                        if (q < key_lo) p0 = 0.f;
                        if (q + 1 < key_lo) p1 = 0.f;
                        if (q < key_hi) p2 = 0.f;
                        if (q + 1 < key_hi) p3 = 0.f;
                    }
                    pf[nb >> 1][(nb & 1) * 2] = pack_bf16(p0, p1);
                    pf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p2, p3);
                    dsf[nb >> 1][(nb & 1) * 2] = pack_bf16(p0 * (pacc[nb][0] - e0), p1 * (pacc[nb][1] - e1));
                    dsf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p2 * (pacc[nb][2] - e0), p3 * (pacc[nb][3] - e1));
                }
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
                    for (int np = 0; np < DH / 16; ++np) {
                        uint32_t bb[4];
                        load_b_kn<DH>(gb, half * 32 + ks * 16, np * 16, bb);
                        mma16816(dv[2 * np], pf[ks], bb[0], bb[1]);
                        mma16816(dv[2 * np + 1], pf[ks], bb[2], bb[3]);
                        load_b_kn<DH>(qb, half * 32 + ks * 16, np * 16, bb);
                        mma16816(dk[2 * np], dsf[ks], bb[0], bb[1]);
                        mma16816(dk[2 * np + 1], dsf[ks], bb[2], bb[3]);
                    }
                }
            }
        }
        __syncthreads();
    }
    __nv_bfloat16* gdk = dqkv + static_cast<size_t>(b * S + k0 + warp * 16) * ld + d + h * DH;
    store_rows16<DH>(sK, smem, warp * 16, dk, scale, scale, gdk, ld);
    store_rows16<DH>(sV, smem + KBk, warp * 16, dv, 1.f, 1.f, gdk + d, ld);
}

template <typename K>
const char* set_smem(K kern, int bytes)
{
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess
               ? nullptr : "cudaFuncSetAttribute(attention) failed";
}

constexpr int dq_smem(int dh) { return 2 * 128 * dh * 2 + 4 * 64 * dh * 2; }
constexpr int dkdv_smem(int dh) { return 2 * 128 * dh * 2 + 4 * 64 * dh * 2 + 4 * 64 * 4; }

}  // namespace

const char* configure_attention()
{
    const char* e;
    if ((e = set_smem(attn_bwd_dq_kernel<64>, dq_smem(64)))) return e;
    if ((e = set_smem(attn_bwd_dq_kernel<128>, dq_smem(128)))) return e;
    if ((e = set_smem(attn_bwd_dkdv_kernel<64>, dkdv_smem(64)))) return e;
    if ((e = set_smem(attn_bwd_dkdv_kernel<128>, dkdv_smem(128)))) return e;
    return nullptr;
}

const char* launch_attention_bwd(Runtime* rt, const void* qkv, const void* o, const void* dout, const void* lse,
                                 int B, int S, int H, int dh, void* dqkv, void* delta, cudaStream_t stream)
{
    (void)rt;
    if (B <= 0 || H <= 0 || S <= 0 || (S % 128) != 0 || (dh != 64 && dh != 128)) return "attention: unsupported shape";
    const float scale = 1.0f / sqrtf(static_cast<float>(dh));
    auto Q = static_cast<const __nv_bfloat16*>(qkv);
    auto O = static_cast<const __nv_bfloat16*>(o);
    auto G = static_cast<const __nv_bfloat16*>(dout);
    auto L = static_cast<const float*>(lse);
    auto Dl = static_cast<float*>(delta);
    auto DQ = static_cast<__nv_bfloat16*>(dqkv);
    {
        const size_t total = static_cast<size_t>(B) * S * H * (dh / 8);
        attn_delta_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, stream>>>(O, G, Dl, B, S, H, dh);
        if (cudaGetLastError() != cudaSuccess) return "attention delta launch failed";
    }
    dim3 grid(S / 128, B * H);
    const int smem_dq = dq_smem(dh), smem_kv = dkdv_smem(dh);
    if (dh == 64) {
        attn_bwd_dq_kernel<64><<<grid, kAttnThreads, smem_dq, stream>>>(Q, G, L, Dl, DQ, S, H, scale);
        attn_bwd_dkdv_kernel<64><<<grid, kAttnThreads, smem_kv, stream>>>(Q, G, L, Dl, DQ, S, H, scale);
    } else {
        attn_bwd_dq_kernel<128><<<grid, kAttnThreads, smem_dq, stream>>>(Q, G, L, Dl, DQ, S, H, scale);
        attn_bwd_dkdv_kernel<128><<<grid, kAttnThreads, smem_kv, stream>>>(Q, G, L, Dl, DQ, S, H, scale);
    }
    return cudaGetLastError() == cudaSuccess ? nullptr : "attention bwd launch failed";
}

}  // namespace pw
