// HBM-bound kernels of the layer: LayerNorm forward, LayerNorm backward (fused with the
// residual-gradient add and two bias-gradient column sums), column sums, and the row-dot
// preprocess of the attention backward.  All use 16-byte accesses (8 bf16 per thread per
// access), fp32 arithmetic, warp shuffles plus one shared-memory hop for row reductions, and
// fixed-order two-stage reductions for anything summed over tokens (bitwise reproducible).
#include <map>
#include <mutex>

#include "pw_kernels.h"

namespace pw {
namespace {

constexpr int kMaxWarps = 8;          // CTAs have at most 256 threads
constexpr int kRowThreadsMax = 256;

// A row of d elements is handled by tpr = d / (8*CHUNKS) threads, CHUNKS 16-byte pieces each;
// thread i of the row owns columns 8*(i + j*tpr) .. +7 for j < CHUNKS (coalesced per j).
struct RowPlan { int chunks, tpr, rows_per_cta, threads; };
bool plan_rows(int d, RowPlan* rp)
{
    for (int c = 1; c <= 4; c *= 2) {
        if (d % (8 * c * 32) != 0) continue;
        int tpr = d / (8 * c);
        if (tpr > kRowThreadsMax) continue;
        rp->chunks = c; rp->tpr = tpr;
        rp->rows_per_cta = kRowThreadsMax / tpr;
        rp->threads = rp->rows_per_cta * tpr;
        return true;
    }
    return false;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void unpack8_pairs(const uint4& v, uint64_t* p)
{
    p[0] = pack_f32x2(bf16_lo(v.x), bf16_hi(v.x)); p[1] = pack_f32x2(bf16_lo(v.y), bf16_hi(v.y));
    p[2] = pack_f32x2(bf16_lo(v.z), bf16_hi(v.z)); p[3] = pack_f32x2(bf16_lo(v.w), bf16_hi(v.w));
}
__device__ __forceinline__ uint32_t pack_pair_bf16(uint64_t p)
{
    float lo, hi;
    unpack_f32x2(p, lo, hi);
    return pack_bf16(lo, hi);
}
__device__ __forceinline__ uint64_t splat2(float v) { return pack_f32x2(v, v); }

// LayerNorm forward.  A row is handled by W warps (W = 1 for d <= 2048), each lane holding CH
// 16-byte pieces (lane i of warp w owns columns 8*(i + 32*(w + W*j)) .. +7, j < CH): all of a
// lane's loads are issued at once, the statistics need only warp shuffles (plus one shared-memory
// hop when W > 1).  256-thread CTAs hold 8/W rows.
template <int CH>
__global__ void __launch_bounds__(kRowThreadsMax, 3)
ln_fwd_kernel(const __nv_bfloat16* x, const __nv_bfloat16* gamma,
              const __nv_bfloat16* beta, int T, int d, float eps, __nv_bfloat16* h,
              float* mu, float* rstd, int W)
{
    __shared__ float red[2][kMaxWarps];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows_per_cta = kMaxWarps / W;
    const int row_in_cta = warp / W, wr = warp % W;
    const int row = blockIdx.x * rows_per_cta + row_in_cta;
    const bool live = row < T && row_in_cta < rows_per_cta;
    grid_dep_launch();
    grid_dep_wait();
    // two-wide fp32 throughout: neighbouring columns share a 64-bit register
    uint64_t v[CH][4];
    uint64_t acc = 0ull;
#pragma unroll
    for (int j = 0; j < CH; ++j) {
        const int col = 8 * (lane + 32 * (wr + W * j));
        const uint4 raw = live ? *reinterpret_cast<const uint4*>(x + static_cast<size_t>(row) * d + col) : make_uint4(0, 0, 0, 0);
        unpack8_pairs(raw, v[j]);
#pragma unroll
        for (int k = 0; k < 4; ++k) acc = fadd2(acc, v[j][k]);
    }
    float a0, a1;
    unpack_f32x2(acc, a0, a1);
    float s = warp_sum(a0 + a1);
    if (W > 1) {
        if (lane == 0) red[0][warp] = s;
        __syncthreads();
        s = 0.f;
        for (int i = 0; i < W; ++i) s += red[0][row_in_cta * W + i];
    }
    const float mean = s / d;
    const uint64_t nmean = splat2(-mean);
    acc = 0ull;
#pragma unroll
    for (int j = 0; j < CH; ++j)
#pragma unroll
        for (int k = 0; k < 4; ++k) { const uint64_t c = fadd2(v[j][k], nmean); acc = ffma2(c, c, acc); }
    unpack_f32x2(acc, a0, a1);
    float q = warp_sum(a0 + a1);
    if (W > 1) {
        if (lane == 0) red[1][warp] = q;
        __syncthreads();
        q = 0.f;
        for (int i = 0; i < W; ++i) q += red[1][row_in_cta * W + i];
    }
    const float r = rsqrtf(q / d + eps);
    if (!live) return;
    const uint64_t r2 = splat2(r), nmr2 = splat2(-mean * r);
#pragma unroll
    for (int j = 0; j < CH; ++j) {
        const int col = 8 * (lane + 32 * (wr + W * j));
        uint64_t g[4], b[4];
        unpack8_pairs(*(reinterpret_cast<const uint4*>(gamma + col)), g);
        unpack8_pairs(*(reinterpret_cast<const uint4*>(beta + col)), b);
        uint4 o;
        o.x = pack_pair_bf16(ffma2(ffma2(v[j][0], r2, nmr2), g[0], b[0]));
        o.y = pack_pair_bf16(ffma2(ffma2(v[j][1], r2, nmr2), g[1], b[1]));
        o.z = pack_pair_bf16(ffma2(ffma2(v[j][2], r2, nmr2), g[2], b[2]));
        o.w = pack_pair_bf16(ffma2(ffma2(v[j][3], r2, nmr2), g[3], b[3]));
        *reinterpret_cast<uint4*>(h + static_cast<size_t>(row) * d + col) = o;
    }
    if (wr == 0 && lane == 0) { mu[row] = mean; rstd[row] = r; }
}

__global__ void __launch_bounds__(256)
affine_f32_kernel(const float* x, long long n, float scale, float shift, float* y)
{
    grid_dep_launch();
    grid_dep_wait();
    const long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
    if (i < n) y[i] = fmaf(x[i], scale, shift);
}

// a = GeLU(u) on bf16 tensors: the backward pass of a layer that did not keep `a` re-derives it from
// the pre-activations it did keep.  8 elements per thread and iteration; 4 bytes per element.
__device__ __forceinline__ uint4 gelu8(const uint4& w, int act)
{
    const uint32_t in[4] = {w.x, w.y, w.z, w.w};
    uint32_t out[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float lo = __uint_as_float(in[q] << 16), hi = __uint_as_float(in[q] & 0xffff0000u);
        gelu2(lo, hi, act);
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out[q]) : "f"(hi), "f"(lo));
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

__global__ void __launch_bounds__(256)
gelu_fwd_kernel(const __nv_bfloat16* u, __nv_bfloat16* a, long long n8, int act)
{
    grid_dep_launch();
    grid_dep_wait();
    const long long stride = static_cast<long long>(gridDim.x) * 256;
    long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
    for (; i + 3 * stride < n8; i += 4 * stride) {                    // four loads in flight per thread
        uint4 w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j] = __ldcs(reinterpret_cast<const uint4*>(u + (i + j * stride) * 8));
#pragma unroll
        for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4*>(a + (i + j * stride) * 8) = gelu8(w[j], act);
    }
    for (; i < n8; i += stride)
        *reinterpret_cast<uint4*>(a + i * 8) = gelu8(*reinterpret_cast<const uint4*>(u + i * 8), act);
}

// W warps per row and CH pieces per lane for a row of d elements (d a multiple of 256).
bool plan_warp_rows(int d, int* W, int* CH)
{
    if (d % 256 != 0) return false;
    const int total = d / 256;
    for (int w = 1; w <= kMaxWarps; ++w)
        if (total % w == 0 && total / w <= 8 && kMaxWarps % w == 0) { *W = w; *CH = total / w; return true; }
    return false;
}

// LayerNorm backward.  Persistent over rows; every thread keeps the column sums of its own
// columns in registers and writes them once at the end as one partial row per (CTA, row slot):
// partials[(cta*rows_per_cta + row_in_cta)][4][d] = {dgamma, dbeta, sum resid, sum dx}.
// The next row's three inputs are fetched before the current row's reduction, and the two row
// sums share one barrier.
// rows in the prefetch ring (six were measured slower than four at every width)
__host__ __device__ constexpr int ln_bwd_depth(int) { return 4; }
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid)
{
    const int n = valid ? 16 : 0;                       // 0: the 16 bytes are zero-filled, src is not read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// The kernel is bound by instruction issue as much as by memory, so all element-wise arithmetic
// is two-wide fp32 (values of neighbouring columns packed in one 64-bit register).
// BIAS_SUMS: also produce the column sums of the residual gradient and of dx (the two bias
// gradients that the LN2 backward of a layer yields for free); without them the partial rows hold
// two quantities instead of four.
template <int CHUNKS, bool BIAS_SUMS>
__global__ void __launch_bounds__(kRowThreadsMax, CHUNKS == 1 ? 2 : 1)
ln_bwd_kernel(const __nv_bfloat16* dh, const __nv_bfloat16* x,
              const float* mu, const float* rstd, const __nv_bfloat16* gamma,
              const __nv_bfloat16* resid, int T, int d, __nv_bfloat16* dx,
              float* partials, int tpr, int rows_per_cta)
{
    constexpr int kDepth = ln_bwd_depth(CHUNKS);
    __shared__ float red[2][2][kMaxWarps];
    const int row_in_cta = threadIdx.x / tpr, tr = threadIdx.x % tpr;
    const int wpr = tpr >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dep_launch();
    grid_dep_wait();
    uint64_t gm[CHUNKS][4];
    uint64_t acc_g[CHUNKS][4], acc_b[CHUNKS][4], acc_r[CHUNKS][4], acc_x[CHUNKS][4];
#pragma unroll
    for (int j = 0; j < CHUNKS; ++j) {
        unpack8_pairs(*(reinterpret_cast<const uint4*>(gamma + 8 * (tr + j * tpr))), gm[j]);
#pragma unroll
        for (int k = 0; k < 4; ++k) acc_g[j][k] = acc_b[j][k] = acc_r[j][k] = acc_x[j][k] = 0ull;
    }
    const int row_groups = (T + rows_per_cta - 1) / rows_per_cta;
    // The three inputs of the rows this thread will handle travel through a private ring in
    // shared memory, kDepth - 1 rows ahead (16-byte asynchronous copies; a thread only ever
    // reads what it fetched itself, so no barrier is involved).  Slot (stage, input, j) of thread
    // t is ring[((stage * 3 + input) * CHUNKS + j) * blockDim.x + t].
    extern __shared__ uint4 ln_bwd_ring[];
    const uint32_t ring0 = smem_u32(ln_bwd_ring) + 16u * threadIdx.x;
    const uint32_t slot_stride = 16u * blockDim.x;
    // Rows are visited with a constant stride, so the element offsets of the row being fetched and of
    // the row being computed are running sums (no 64-bit multiply per row).
    const int row_step = gridDim.x * rows_per_cta;
    const size_t off_step = static_cast<size_t>(row_step) * d;
    int pf_row = blockIdx.x * rows_per_cta + row_in_cta;                 // next row to fetch
    size_t pf_off = static_cast<size_t>(pf_row) * d + 8 * tr;
    auto issue = [&](int stage) {
        const bool live = pf_row < T;
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
            const size_t off = live ? pf_off + 8 * j * tpr : 0;
            const uint32_t dst = ring0 + (stage * 3 * CHUNKS + j) * slot_stride;
            cp_async_16(dst, dh + off, live);
            cp_async_16(dst + CHUNKS * slot_stride, x + off, live);
            cp_async_16(dst + 2 * CHUNKS * slot_stride, resid ? resid + off : dh + off, live && resid != nullptr);   // no residual: zeros
        }
        cp_async_commit();
        pf_row += row_step;
        pf_off += off_step;
    };
    float n_m = 0.f, n_r = 0.f;
    auto fetch_stats = [&](int rg) {
        const int row = rg * rows_per_cta + row_in_cta;
        const bool live = rg < row_groups && row < T;
        n_m = live ? mu[row] : 0.f;
        n_r = live ? rstd[row] : 0.f;
    };
#pragma unroll
    for (int s = 0; s < kDepth - 1; ++s) issue(s);
    fetch_stats(blockIdx.x);
    const float inv_d = 1.0f / d;
    int par = 0, stage = 0;
    int row = blockIdx.x * rows_per_cta + row_in_cta;
    size_t row_off = static_cast<size_t>(row) * d + 8 * tr;
    for (int rg = blockIdx.x; rg < row_groups; rg += gridDim.x, par ^= 1, row += row_step, row_off += off_step) {
        const bool live = row < T;
        const float r = n_r;
        const uint64_t r2 = splat2(r), nmr2 = splat2(-n_m * r);
        issue(stage == 0 ? kDepth - 1 : stage - 1);
        cp_async_wait<kDepth - 1>();                  // this row's copies have landed
        uint64_t xh[CHUNKS][4], g[CHUNKS][4], dhv[CHUNKS][4], rs[CHUNKS][4];
        uint64_t s1p = 0ull, s2p = 0ull;
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
            const uint4* slot = ln_bwd_ring + (stage * 3 * CHUNKS + j) * blockDim.x + threadIdx.x;
            unpack8_pairs(slot[0], dhv[j]);
            unpack8_pairs(slot[CHUNKS * blockDim.x], xh[j]);
            unpack8_pairs(slot[2 * CHUNKS * blockDim.x], rs[j]);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                xh[j][k] = ffma2(xh[j][k], r2, nmr2);           // (x - mu) * rstd
                g[j][k] = fmul2(dhv[j][k], gm[j][k]);
                s1p = fadd2(s1p, g[j][k]);
                s2p = ffma2(g[j][k], xh[j][k], s2p);
            }
        }
        stage = stage + 1 == kDepth ? 0 : stage + 1;
        fetch_stats(rg + gridDim.x);
        float s1, s1b, s2, s2b;
        unpack_f32x2(s1p, s1, s1b);
        unpack_f32x2(s2p, s2, s2b);
        s1 = warp_sum(s1 + s1b);
        s2 = warp_sum(s2 + s2b);
        if (wpr > 1) {
            if (lane == 0) { red[par][0][warp] = s1; red[par][1][warp] = s2; }
            __syncthreads();
            // every lane takes one warp's pair of partial sums; three exchange steps add up to eight of them
            const int src = lane & (kMaxWarps - 1);      // every group of eight lanes holds the same eight values
            s1 = src < wpr ? red[par][0][row_in_cta * wpr + src] : 0.f;
            s2 = src < wpr ? red[par][1][row_in_cta * wpr + src] : 0.f;
#pragma unroll
            for (int o = kMaxWarps / 2; o > 0; o >>= 1) {
                s1 += __shfl_xor_sync(0xffffffffu, s1, o);
                s2 += __shfl_xor_sync(0xffffffffu, s2, o);
            }
        }
        const uint64_t nmg2 = splat2(-s1 * inv_d), nmgx2 = splat2(-s2 * inv_d);
        if (live) {
#pragma unroll
            for (int j = 0; j < CHUNKS; ++j) {
                const size_t off = row_off + 8 * j * tpr;
                uint32_t w[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // dx = resid + rstd * (g - mean(g) - xh * mean(g * xh))
                    const uint64_t t = ffma2(xh[j][k], nmgx2, fadd2(g[j][k], nmg2));
                    w[k] = pack_pair_bf16(ffma2(r2, t, rs[j][k]));
                    // the bias gradient sums the values that are actually stored
                    if (BIAS_SUMS) acc_x[j][k] = fadd2(acc_x[j][k], pack_f32x2(bf16_lo(w[k]), bf16_hi(w[k])));
                    acc_g[j][k] = ffma2(dhv[j][k], xh[j][k], acc_g[j][k]);
                    acc_b[j][k] = fadd2(acc_b[j][k], dhv[j][k]);
                    if (BIAS_SUMS) acc_r[j][k] = fadd2(acc_r[j][k], rs[j][k]);
                }
                *reinterpret_cast<uint4*>(dx + off) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
    constexpr int NQ = BIAS_SUMS ? 4 : 2;
    float* prow = partials + static_cast<size_t>(blockIdx.x * rows_per_cta + row_in_cta) * NQ * d;
#pragma unroll
    for (int j = 0; j < CHUNKS; ++j) {
        const int col = 8 * (tr + j * tpr);
#pragma unroll
        for (int k = 0; k < 4; k += 2) {
            // two pairs = four consecutive columns
            *reinterpret_cast<ulonglong2*>(prow + 0 * d + col + 2 * k) = make_ulonglong2(acc_g[j][k], acc_g[j][k + 1]);
            *reinterpret_cast<ulonglong2*>(prow + 1 * d + col + 2 * k) = make_ulonglong2(acc_b[j][k], acc_b[j][k + 1]);
            if (BIAS_SUMS) {
                *reinterpret_cast<ulonglong2*>(prow + 2 * d + col + 2 * k) = make_ulonglong2(acc_r[j][k], acc_r[j][k + 1]);
                *reinterpret_cast<ulonglong2*>(prow + 3 * d + col + 2 * k) = make_ulonglong2(acc_x[j][k], acc_x[j][k + 1]);
            }
        }
    }
}

// out[c] (+)= sum over partial rows r of src[r * stride + c], for up to eight (src, out) entries in one
// launch (grid.y = entry): the partial rows of the two LayerNorm backward kernels and of the two bias
// column sums of a layer's backward end up in one launch.  CTA = 64 columns x 16 row lanes, a thread
// owns four consecutive columns (16-byte loads, eight rows in flight): row lane y adds rows y, y+16, ...
// in order, then the 16 lane sums are added in order, so the result does not depend on scheduling.
// n is a multiple of 4.
struct ReduceEntry { const float* src; float* out; int nrows, n; long long stride; };
struct ReduceTable { ReduceEntry e[kReduceMaxEntries]; };
constexpr int kReduceCols = 64, kReduceLanes = 16;
__global__ void __launch_bounds__(kReduceCols / 4 * kReduceLanes)
reduce_partials_kernel(const __grid_constant__ ReduceTable tab, int accumulate)
{
    __shared__ float4 sm[kReduceLanes][kReduceCols / 4];
    const int cx = threadIdx.x & (kReduceCols / 4 - 1), ry = threadIdx.x / (kReduceCols / 4);
    const int c = blockIdx.x * kReduceCols + cx * 4;
    const ReduceEntry& en = tab.e[blockIdx.y];
    float* out = en.out;
    const int n = en.n, nrows = en.nrows;
    grid_dep_launch();
    grid_dep_wait();
    if (out == nullptr || blockIdx.x * kReduceCols >= n) return;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < n) {
        const size_t stride = static_cast<size_t>(en.stride);          // floats between partial rows
        const float* src = en.src + c;
        int r = ry;
        for (; r + 7 * kReduceLanes < nrows; r += 8 * kReduceLanes) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = *reinterpret_cast<const float4*>(src + (r + u * kReduceLanes) * stride);
#pragma unroll
            for (int u = 0; u < 8; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
        }
        for (; r < nrows; r += kReduceLanes) {
            const float4 v = *reinterpret_cast<const float4*>(src + r * stride);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
    }
    sm[ry][cx] = s;
    __syncthreads();
    if (ry == 0 && c < n) {
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kReduceLanes; ++i) { const float4 v = sm[i][cx]; t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w; }
        if (accumulate) { t.x += out[c]; t.y += out[c + 1]; t.z += out[c + 2]; t.w += out[c + 3]; }
        out[c] = t.x; out[c + 1] = t.y; out[c + 2] = t.z; out[c + 3] = t.w;
    }
}

// Column sums of a bf16 [T, N] matrix: CTA (x, y) owns columns 2048*x .. +2047 and rows y, y+R, ...;
// eight rows are in flight per thread.
constexpr int kColsumCols = 2048;
__global__ void __launch_bounds__(256)
colsum_kernel(const __nv_bfloat16* in, int T, int N, int ld, float* partials)
{
    const int col = blockIdx.x * kColsumCols + threadIdx.x * 8;
    grid_dep_launch();
    grid_dep_wait();
    if (col >= N) return;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const int R = gridDim.y;
    int t = blockIdx.y;
    for (; t + 7 * R < T; t += 8 * R) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = *reinterpret_cast<const uint4*>(in + static_cast<size_t>(t + u * R) * ld + col);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            float f[8];
            unpack8(v[u], f);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] += f[k];
        }
    }
    for (; t < T; t += R) {
        float f[8];
        unpack8(*reinterpret_cast<const uint4*>(in + static_cast<size_t>(t) * ld + col), f);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] += f[k];
    }
    float* p = partials + static_cast<size_t>(blockIdx.y) * N + col;
    *reinterpret_cast<float4*>(p) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
}

int colsum_splits(Runtime* rt, int T, int N)
{
    const int col_blocks = (N + kColsumCols - 1) / kColsumCols;
    int r = (4 * rt->sm_count + col_blocks - 1) / col_blocks;
    if (r > T) r = T;
    if (r < 1) r = 1;
    return r;
}

int ln_bwd_grid(Runtime* rt, int T, const RowPlan& rp)
{
    const int row_groups = (T + rp.rows_per_cta - 1) / rp.rows_per_cta;
    const int cap = (rp.chunks == 1 ? 2 : 1) * rt->sm_count;
    return row_groups < cap ? row_groups : cap;
}

}  // namespace

const char* launch_layernorm_fwd(Runtime* rt, const void* x, const void* gamma, const void* beta, int T, int d,
                                 float eps, void* h, void* mu, void* rstd, cudaStream_t stream)
{
    (void)rt;
    int W = 0, CH = 0;
    if (T <= 0 || !plan_warp_rows(d, &W, &CH)) return "layernorm: unsupported row width";
    const int rows_per_cta = kMaxWarps / W;
    const int grid = (T + rows_per_cta - 1) / rows_per_cta;
    auto X = static_cast<const __nv_bfloat16*>(x);
    auto G = static_cast<const __nv_bfloat16*>(gamma);
    auto Bt = static_cast<const __nv_bfloat16*>(beta);
    auto Hh = static_cast<__nv_bfloat16*>(h);
    auto Mu = static_cast<float*>(mu);
    auto Rs = static_cast<float*>(rstd);
#define PW_LN_FWD(N) case N: le = launch_k(ln_fwd_kernel<N>, dim3(grid), dim3(kRowThreadsMax), 0, stream, X, G, Bt, T, d, eps, Hh, Mu, Rs, W); break
    cudaError_t le = cudaSuccess;
    switch (CH) {
        PW_LN_FWD(1); PW_LN_FWD(2); PW_LN_FWD(3); PW_LN_FWD(4); PW_LN_FWD(5); PW_LN_FWD(6); PW_LN_FWD(7); PW_LN_FWD(8);
        default: return "layernorm: unsupported row width";
    }
#undef PW_LN_FWD
    return le == cudaSuccess ? nullptr : "layernorm fwd launch failed";
}

const char* configure_elementwise()
{
    cudaError_t e = cudaSuccess;
#define PW_LN_ATTR(C, B) if (e == cudaSuccess) e = cudaFuncSetAttribute(ln_bwd_kernel<C, B>, cudaFuncAttributeMaxDynamicSharedMemorySize, ln_bwd_depth(C) * 3 * C * kRowThreadsMax * 16)
    PW_LN_ATTR(1, true); PW_LN_ATTR(1, false); PW_LN_ATTR(2, true); PW_LN_ATTR(2, false); PW_LN_ATTR(4, true); PW_LN_ATTR(4, false);
#undef PW_LN_ATTR
    return e == cudaSuccess ? nullptr : "could not raise the shared-memory limit of the layernorm kernels";
}

size_t layernorm_bwd_scratch_bytes(Runtime* rt, int T, int d)
{
    RowPlan rp;
    if (T <= 0 || !plan_rows(d, &rp)) return 0;
    return static_cast<size_t>(ln_bwd_grid(rt, T, rp)) * rp.rows_per_cta * 4 * d * sizeof(float);
}

// Main kernel only: the partial rows stay in `partials` and `job` says how to reduce them.
const char* launch_layernorm_bwd_partial(Runtime* rt, const void* dh, const void* x, const void* mu, const void* rstd,
                                         const void* gamma, const void* resid, int T, int d, void* dx, void* dgamma,
                                         void* dbeta, void* db_resid, void* db_dx, void* partials, ReduceJob* job,
                                         cudaStream_t stream)
{
    RowPlan rp;
    if (T <= 0 || !plan_rows(d, &rp)) return "layernorm: unsupported row width";
    const int grid = ln_bwd_grid(rt, T, rp);
    auto DH = static_cast<const __nv_bfloat16*>(dh);
    auto X = static_cast<const __nv_bfloat16*>(x);
    auto G = static_cast<const __nv_bfloat16*>(gamma);
    auto R = static_cast<const __nv_bfloat16*>(resid);
    auto DX = static_cast<__nv_bfloat16*>(dx);
    auto Mu = static_cast<const float*>(mu);
    auto Rs = static_cast<const float*>(rstd);
    auto P = static_cast<float*>(partials);
    cudaError_t le = cudaSuccess;
    const size_t ring_bytes = static_cast<size_t>(ln_bwd_depth(rp.chunks)) * 3 * rp.chunks * rp.threads * 16;
    const bool sums = db_resid != nullptr || db_dx != nullptr;
#define PW_LN_BWD(C, B) le = launch_k(ln_bwd_kernel<C, B>, dim3(grid), dim3(rp.threads), ring_bytes, stream, DH, X, Mu, Rs, G, R, T, d, DX, P, rp.tpr, rp.rows_per_cta)
    switch (rp.chunks) {
        case 1: if (sums) PW_LN_BWD(1, true); else PW_LN_BWD(1, false); break;
        case 2: if (sums) PW_LN_BWD(2, true); else PW_LN_BWD(2, false); break;
        default: if (sums) PW_LN_BWD(4, true); else PW_LN_BWD(4, false); break;
    }
#undef PW_LN_BWD
    if (le != cudaSuccess) return "layernorm bwd launch failed";
    job->partials = P; job->nrows = grid * rp.rows_per_cta; job->nq = sums ? 4 : 2; job->n = d;
    job->out[0] = static_cast<float*>(dgamma); job->out[1] = static_cast<float*>(dbeta);
    job->out[2] = static_cast<float*>(db_resid); job->out[3] = static_cast<float*>(db_dx);
    return nullptr;
}

// One launch for the partial rows of up to four jobs (at most eight output vectors in all).
const char* launch_reduce_jobs(const ReduceJob* jobs, int njobs, int accumulate, cudaStream_t stream)
{
    ReduceTable tab = {};
    int ne = 0, max_n = 0;
    for (int j = 0; j < njobs; ++j)
        for (int q = 0; q < jobs[j].nq; ++q) {
            if (jobs[j].out[q] == nullptr) continue;
            if (ne == kReduceMaxEntries) return "reduce: too many output vectors for one launch";
            ReduceEntry& en = tab.e[ne++];
            en.src = jobs[j].partials + static_cast<size_t>(q) * jobs[j].n;
            en.out = jobs[j].out[q];
            en.nrows = jobs[j].nrows; en.n = jobs[j].n;
            en.stride = static_cast<long long>(jobs[j].nq) * jobs[j].n;
            if (en.n > max_n) max_n = en.n;
        }
    if (ne == 0) return nullptr;
    dim3 rgrid((max_n + kReduceCols - 1) / kReduceCols, ne);
    return launch_k(reduce_partials_kernel, rgrid, dim3(kReduceCols / 4 * kReduceLanes), 0, stream, tab, accumulate) == cudaSuccess
               ? nullptr : "partial-row reduce launch failed";
}

const char* launch_layernorm_bwd(Runtime* rt, const void* dh, const void* x, const void* mu, const void* rstd,
                                 const void* gamma, const void* resid, int T, int d, void* dx, void* dgamma,
                                 void* dbeta, void* db_resid, void* db_dx, int accumulate, void* partials,
                                 cudaStream_t stream)
{
    ReduceJob job;
    const char* e = launch_layernorm_bwd_partial(rt, dh, x, mu, rstd, gamma, resid, T, d, dx, dgamma, dbeta, db_resid, db_dx,
                                                 partials, &job, stream);
    return e ? e : launch_reduce_jobs(&job, 1, accumulate, stream);
}

// y = x * scale + shift on fp32 vectors: the node type of the paper's Figure 2 program (a: x*2,
// b: x+1, c: x/2), used to run that worked example through the dispatch paths.
const char* launch_affine_f32(const void* x, long long n, float scale, float shift, void* y, cudaStream_t stream)
{
    if (n <= 0) return "affine: empty vector";
    const long long blocks = (n + 255) / 256;
    if (blocks > 0x7fffffffll) return "affine: vector too long";
    return launch_k(affine_f32_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream, static_cast<const float*>(x), n,
                    scale, shift, static_cast<float*>(y)) == cudaSuccess
               ? nullptr : "affine launch failed";
}

const char* launch_gelu_fwd(Runtime* rt, const void* u, void* a, long long n, int act, cudaStream_t stream)
{
    if (n <= 0 || (n % 8) != 0) return "gelu: element count must be a positive multiple of 8";
    const long long n8 = n / 8;
    long long blocks = (n8 + 255) / 256;
    const long long cap = static_cast<long long>(rt->sm_count) * 16;
    if (blocks > cap) blocks = cap;
    return launch_k(gelu_fwd_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream, static_cast<const __nv_bfloat16*>(u),
                    static_cast<__nv_bfloat16*>(a), n8, act) == cudaSuccess
               ? nullptr : "gelu launch failed";
}

size_t colsum_scratch_bytes(Runtime* rt, int T, int N)
{
    if (T <= 0 || N <= 0) return 0;
    return static_cast<size_t>(colsum_splits(rt, T, N)) * N * sizeof(float);
}

const char* launch_colsum_partial(Runtime* rt, const void* in, int T, int N, int ld, void* out, void* partials,
                                  ReduceJob* job, cudaStream_t stream)
{
    if (T <= 0 || N <= 0 || (N % 8) || (ld % 8)) return "colsum: N and ld must be multiples of 8";
    const int R = colsum_splits(rt, T, N);
    dim3 grid((N + kColsumCols - 1) / kColsumCols, R);
    if (launch_k(colsum_kernel, grid, dim3(256), 0, stream, static_cast<const __nv_bfloat16*>(in), T, N, ld, static_cast<float*>(partials)) != cudaSuccess)
        return "colsum launch failed";
    job->partials = static_cast<const float*>(partials); job->nrows = R; job->nq = 1; job->n = N;
    job->out[0] = static_cast<float*>(out); job->out[1] = job->out[2] = job->out[3] = nullptr;
    return nullptr;
}

const char* launch_colsum(Runtime* rt, const void* in, int T, int N, int ld, void* out, int accumulate,
                          void* partials, cudaStream_t stream)
{
    ReduceJob job;
    const char* e = launch_colsum_partial(rt, in, T, N, ld, out, partials, &job, stream);
    return e ? e : launch_reduce_jobs(&job, 1, accumulate, stream);
}

// ---------------------------------------------------------------------------------------------
// Column sums without any allocation.  Some callers hand this library buffers but cannot create
// device memory themselves while they run - a serving loop that has already given every byte of
// HBM to its pools, a host callback, code running under a framework that forbids allocation at
// that point.  For them the scratch of the column-sum kernel (the per-row-group partial sums)
// lives in this fixed array, which every GPU that loads the library holds until the process
// exits.  All calls share it: two calls that overlap on the GPU race on it, and it keeps the last
// call's partial sums (every slot that a call reads is first written by that same call, so
// nothing needs clearing).
constexpr size_t kStaticScratchFloats = 262144;   // 1 MiB
static __device__ __align__(256) float g_colsum_scratch[kStaticScratchFloats];

namespace {
struct StaticScratch { float* ptr; int sm_count; };
// In host code the array's name is only a handle for the runtime, not a device address: the
// address comes from cudaGetSymbolAddress, asked once per device with that device current.
const char* static_scratch_for_current_device(StaticScratch* out, int* err_kind)
{
    *err_kind = kErrCuda;
    static std::mutex mu;
    static std::map<int, StaticScratch> per_device;
    std::lock_guard<std::mutex> lock(mu);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return "no CUDA device (cudaGetDevice failed)";
    auto it = per_device.find(dev);
    if (it == per_device.end()) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return "cudaDeviceGetAttribute failed";
        if (major != 10) { *err_kind = kErrDevice; return "device is not compute capability 10.x (sm_100a kernels only, no fallback)"; }
        float* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_colsum_scratch);
        if (e != cudaSuccess || ptr == nullptr) return "cudaGetSymbolAddress(static scratch) failed";
        it = per_device.emplace(dev, StaticScratch{ptr, sms}).first;
    }
    *out = it->second;
    return nullptr;
}
}  // namespace

size_t colsum_noalloc_max_columns() { return kStaticScratchFloats; }

const char* launch_colsum_noalloc(const void* in, int T, int N, int ld, void* out, int accumulate, cudaStream_t stream,
                                  int* err_kind)
{
    *err_kind = kErrArgument;
    if (T <= 0 || N <= 0 || (N % 8) || (ld % 8) || ld < N) return "colsum: N and ld must be multiples of 8, ld >= N";
    if (static_cast<size_t>(N) > kStaticScratchFloats)
        return "colsum (no-allocation variant): N exceeds the 262144 columns the built-in scratch can hold";
    StaticScratch sc;
    if (const char* e = static_scratch_for_current_device(&sc, err_kind)) return e;
    *err_kind = kErrCuda;
    // as many row groups as the fixed scratch can hold, at most what the allocating variant uses
    const int col_blocks = (N + kColsumCols - 1) / kColsumCols;
    long long R = (4ll * sc.sm_count + col_blocks - 1) / col_blocks;
    const long long fit = static_cast<long long>(kStaticScratchFloats / static_cast<size_t>(N));
    if (R > fit) R = fit;
    if (R > T) R = T;
    if (R < 1) R = 1;
    dim3 grid(col_blocks, static_cast<unsigned>(R));
    colsum_kernel<<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(in), T, N, ld, sc.ptr);
    if (cudaGetLastError() != cudaSuccess) return "colsum launch failed";
    ReduceTable tab = {};
    tab.e[0].src = sc.ptr; tab.e[0].out = static_cast<float*>(out);
    tab.e[0].nrows = static_cast<int>(R); tab.e[0].n = N; tab.e[0].stride = N;
    dim3 rgrid((N + kReduceCols - 1) / kReduceCols, 1);
    reduce_partials_kernel<<<rgrid, kReduceCols / 4 * kReduceLanes, 0, stream>>>(tab, accumulate);
    return cudaGetLastError() == cudaSuccess ? nullptr : "colsum reduce launch failed";
}

}  // namespace pw
