// One decoder layer's forward, or its backward, as ONE cooperative launch, for calls so small
// (workload 1: 256 tokens, width 256, 1.2 GFLOP forward + backward) that launches, ramps and
// hand-offs between kernels set the time, not arithmetic: the regime of the dispatch study of
// Section 5.1 (Figures 5 and 6), where a computation is shorter than the cost of issuing it.
//
// The 7 forward / 15 backward launches of the multi-kernel path become 5 / 7 phases of one persistent grid
// (one 256-thread CTA per SM); a phase is a list of independent units (a 64 x 64 output tile of a
// GEMM, a slice of its K range, 64 query or key rows of one head, four LayerNorm rows, 16 columns of
// a bias sum) that the CTAs take round-robin, and phases are separated by a bounded grid barrier.
// Steps that do not depend on one another share a phase (a data-gradient GEMM, the weight-gradient
// GEMM and the bias sum that hang off the same tensor), LayerNorm is applied while a GEMM stages its
// A rows, and rowsum(dO * O) is taken by the attention-backward units themselves.
//
// At these sizes a tile of 64 x 64 keeps 16 ... 144 SMs busy where the 128 x 256 tcgen05 tiles of
// the large-shape kernels would keep 2 ... 8; the products run on mma.sync (m16n8k16, bf16 in, fp32
// accumulate) from shared memory, which is far below the tcgen05 rate and does not matter here.
// Every sum has a fixed order (split-K partial tiles are added by the last-arriving CTA in slice
// order), so results are bit-reproducible.  Tensors, rounding points (bf16 hand-offs) and the saved
// context are those of the multi-kernel path.
#include "pw_kernels.h"

namespace pw {
namespace {

constexpr int kThreads = 256;                        // 8 warps
constexpr int kChunk = 64 * 64 * 2;                 // one 64 x 64 bf16 operand chunk
constexpr int kStages = 5;                            // four 64-wide K blocks in flight: K = 256 is one trip to L2
constexpr int kMaxD = 512;                          // LayerNorm panel: 64 rows of the full width in shared memory
constexpr int kMaxS = 1024;
constexpr int kSmStage = 0;                         // kStages x (A chunk, B chunk); attention: Q/K/V/dO chunks
constexpr int kSmAux = kSmStage + kStages * 2 * kChunk;      // one chunk of an epilogue operand (residual, u)
constexpr int kAccStride = 68;                               // floats per row of the accumulator tile (bank spread)
constexpr int kSmAcc = kSmAux + kChunk;                      // 64 x 64 accumulators on their way to a rolled epilogue loop
constexpr int kSmPanel = kSmAcc + 64 * kAccStride * 4;       // also the lanes of a column-sum unit (16 KB) and the attention merges
constexpr int kSmVec = kSmPanel + 64 * (kMaxD + 8) * 2;     // lse and delta of one (sequence, head)
constexpr int kSmFlag = kSmVec + 2 * kMaxS * 4;
constexpr int kSmBytes = kSmFlag + 16;

constexpr int kSiteBarrier = 900;

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned long long ld_acquire(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long atom_add_acq_rel(unsigned long long* p, unsigned long long v)
{
    unsigned long long old;
    asm volatile("atom.add.acq_rel.gpu.global.u64 %0, [%1], %2;" : "=l"(old) : "l"(p), "l"(v) : "memory");
    return old;
}

// ---------------------------------------------------------------- grid barrier
// One 64-bit arrival counter that only ever grows: arrival number n belongs to barrier n / G and that
// barrier is open once the counter reaches (n / G + 1) G, so one atomic per CTA is the whole
// protocol and the last arrival is itself the release.  Every launch leaves the counter at a multiple
// of G, which is all the next launch (or the replay of a captured graph) needs.  A CTA that waits
// longer than the limit records a timeout in the status word and every CTA leaves.
__device__ bool grid_barrier(unsigned* sync, DeviceStatus* status, int* s_flag)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 1;
        unsigned long long* count = reinterpret_cast<unsigned long long*>(sync);
        const unsigned long long G = gridDim.x;
        const unsigned long long mine = atom_add_acq_rel(count, 1ull);
        const unsigned long long target = (mine / G + 1) * G;
        if (mine + 1 < target) {
            const long long t0 = clock64();
            unsigned spins = 0;
            while (ld_acquire(count) < target) {
                if ((++spins & 0xffu) == 0) {
                    if (*reinterpret_cast<volatile int*>(&status->code) != 0) { ok = 0; break; }
                    if (clock64() - t0 > kWaitCycles) {
                        if (atomicCAS(&status->code, 0, kStatusTimeout) == 0) status->site = kSiteBarrier;
                        ok = 0;
                        break;
                    }
                }
            }
        }
        *s_flag = ok;
    }
    __syncthreads();
    return *s_flag != 0;
}

// ---------------------------------------------------------------- operand chunks in shared memory
// A chunk is 64 rows of 128 bytes; the 16-byte piece c of row r sits at piece c ^ (r & 7), which keeps
// both ldmatrix forms free of bank conflicts.
__device__ __forceinline__ uint32_t swz(int row, int piece) { return row * 128 + ((piece ^ (row & 7)) << 4); }

__device__ __forceinline__ void stage_chunk(uint32_t dst, const uint16_t* src, size_t ld, int tid)
{
#pragma unroll
    for (int i = 0; i < 512 / kThreads; ++i) {
        const int q = tid + i * kThreads, row = q >> 3, piece = q & 7;
        cp_async16(dst + swz(row, piece), src + row * ld + piece * 8);
    }
}
// chunk stored [m or n][k]
__device__ __forceinline__ void frag_a_k(uint32_t base, int r0, int kk, int lane, uint32_t (&a)[4])
{
    ldsm4(base + swz(r0 + (lane & 15), kk * 2 + (lane >> 4)), a);
}
__device__ __forceinline__ void frag_b_k(uint32_t base, int n0, int kk, int lane, uint32_t (&b)[4])
{
    ldsm4(base + swz(n0 + (lane & 7) + ((lane >> 4) << 3), kk * 2 + ((lane >> 3) & 1)), b);
}
// chunk stored [k][m or n]
__device__ __forceinline__ void frag_a_mn(uint32_t base, int m0, int kk, int lane, uint32_t (&a)[4])
{
    ldsm4t(base + swz(kk * 16 + (lane & 7) + ((lane >> 4) << 3), (m0 >> 3) + ((lane >> 3) & 1)), a);
}
__device__ __forceinline__ void frag_b_mn(uint32_t base, int n0, int kk, int lane, uint32_t (&b)[4])
{
    ldsm4t(base + swz(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), (n0 >> 3) + (lane >> 4)), b);
}

// ---------------------------------------------------------------- 64 x 64 output tile, K range [k0, k0 + 64 nk)
// C[m0.., n0..] = sum_k A(m, k) B(k, n).  A_MN: A is stored [K][M] (else [M][K]); B_MN: B is stored
// [K][N] (else [N][K]); A_PANEL: the A rows are already in shared memory (LayerNorm output, full width).
// Warp w owns rows 32 (w & 1) and columns 16 (w >> 1): acc[mi][ni][e] is row 16 mi + lane / 4 + 8 (e / 2),
// column 8 ni + 2 (lane % 4) + e % 2 of that eighth.  prefetch() puts the first chunks in flight, so
// that whatever the unit does before run() (LayerNorm of the A rows, loads of epilogue operands)
// overlaps their way from L2.
template <bool A_MN, bool B_MN, bool A_PANEL>
struct TileGemm {
    const uint16_t* A; size_t lda;
    const uint16_t* Bm; size_t ldb;
    int m0, n0, k0, nk;
    uint32_t stage;

    __device__ __forceinline__ void load(int kc) const
    {
        const int tid = threadIdx.x;
        const uint32_t sa = stage + (kc % kStages) * 2 * kChunk, sb = sa + kChunk;
        const size_t kk0 = k0 + kc * 64;
        if (!A_PANEL) stage_chunk(sa, A_MN ? A + kk0 * lda + m0 : A + m0 * lda + kk0, lda, tid);
        stage_chunk(sb, B_MN ? Bm + kk0 * ldb + n0 : Bm + n0 * ldb + kk0, ldb, tid);
    }
    __device__ __forceinline__ void prefetch() const
    {
#pragma unroll
        for (int s = 0; s < kStages - 1; ++s) {
            if (s < nk) load(s);
            cp_async_commit();
        }
    }
    __device__ __forceinline__ void run(float (&acc)[2][2][4], uint32_t panel, int panel_stride) const
    {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wm = (warp & 1) * 32, wn = (warp >> 1) * 16;
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;
        for (int kc = 0; kc < nk; ++kc) {
            cp_async_wait<kStages - 2>();
            __syncthreads();
            if (kc + kStages - 1 < nk) load(kc + kStages - 1);
            cp_async_commit();
            const uint32_t sa = stage + (kc % kStages) * 2 * kChunk, sb = sa + kChunk;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t af[2][4], bf[4];
#pragma unroll
                for (int mi = 0; mi < 2; ++mi) {
                    if (A_PANEL) {
                        const int row = wm + mi * 16 + (lane & 15), col = k0 + kc * 64 + kk * 16 + (lane >> 4) * 8;
                        ldsm4(panel + row * panel_stride + col * 2, af[mi]);
                    } else if (A_MN) {
                        frag_a_mn(sa, wm + mi * 16, kk, lane, af[mi]);
                    } else {
                        frag_a_k(sa, wm + mi * 16, kk, lane, af[mi]);
                    }
                }
                if (B_MN) frag_b_mn(sb, wn, kk, lane, bf);
                else frag_b_k(sb, wn, kk, lane, bf);
#pragma unroll
                for (int mi = 0; mi < 2; ++mi)
#pragma unroll
                    for (int ni = 0; ni < 2; ++ni) mma16816(acc[mi][ni], af[mi], bf[ni * 2], bf[ni * 2 + 1]);
            }
        }
        cp_async_wait<0>();
        __syncthreads();                                    // the stage buffers may be refilled by the next unit
    }
};

// Split-K: every slice stores its partial tile, the CTA that arrives last adds the slices in slice
// order (its own included, from memory) and returns true: it then runs the epilogue.
__device__ bool splitk_combine(float (&acc)[2][2][4], float* ws, unsigned* sem, int tile, int slice, int nslices, int* s_flag)
{
    if (nslices == 1) return true;
    const int tid = threadIdx.x;
    float* flat = &acc[0][0][0];
    float4* mine = reinterpret_cast<float4*>(ws + static_cast<size_t>(tile * nslices + slice) * 4096);
#pragma unroll
    for (int i = 0; i < 4; ++i) __stcg(mine + i * kThreads + tid, make_float4(flat[4 * i], flat[4 * i + 1], flat[4 * i + 2], flat[4 * i + 3]));
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned prev = atomicAdd(sem + tile, 1u);
        const int last = prev == static_cast<unsigned>(nslices - 1);
        if (last) atomicExch(sem + tile, 0u);
        __threadfence();
        *s_flag = last;
    }
    __syncthreads();
    const bool last = *s_flag != 0;
    __syncthreads();                                        // everyone has read the flag before it is written again
    if (!last) return false;
#pragma unroll
    for (int i = 0; i < 16; ++i) flat[i] = 0.f;
    for (int s = 0; s < nslices; ++s) {
        const float4* part = reinterpret_cast<const float4*>(ws + static_cast<size_t>(tile * nslices + s) * 4096);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 v = __ldcg(part + i * kThreads + tid);
            flat[4 * i] += v.x; flat[4 * i + 1] += v.y; flat[4 * i + 2] += v.z; flat[4 * i + 3] += v.w;
        }
    }
    return true;
}

__device__ __forceinline__ void store_bf16x2(uint16_t* base, size_t idx, float v0, float v1)
{
    *reinterpret_cast<uint32_t*>(base + idx) = pack_bf16(v0, v1);
}

// ---------------------------------------------------------------- LayerNorm of 64 rows in the panel
// The 64 rows of x come into the panel by cp.async (ln_stage_rows, one commit group) and are normalised
// in place by a short rolled loop - code that runs once per launch is paid for by instruction fetch,
// not by arithmetic.  Warp w owns rows 8 w .. 8 w + 7, four at a time: eight lanes share a row (lane
// % 8 owns the 16-byte pieces lane % 8 + 8 j), so a row sum is three shuffles.  Two-pass statistics
// in fp32, like the stand-alone kernel; h = (x - mean) * rstd * gamma + beta replaces x as bf16 and,
// from the CTA of column tile 0, goes to global memory with mean and rstd for the backward pass.
__device__ __forceinline__ void ln_stage_rows(const uint16_t* x, int d, int m0, uint32_t panel, int stride)
{
    const int per_row = d >> 3;                             // 16-byte pieces per row
#pragma unroll 1
    for (int q = threadIdx.x; q < 64 * per_row; q += kThreads) {
        const int row = q / per_row, piece = q - row * per_row;
        cp_async16(panel + row * stride + piece * 16, x + static_cast<size_t>(m0 + row) * d + piece * 8);
    }
}
template <int NP>
__device__ __forceinline__ void ln_rows_in_panel(const uint16_t* gamma, const uint16_t* beta, float eps, int m0, uint8_t* panel,
                                                 int stride, bool write, uint16_t* h, float* mu, float* rstd)
{
    constexpr int d = 256 * NP, kPieces = 4 * NP;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, sub = lane & 7, rsel = lane >> 3;
    const float inv_d = 1.0f / d;
    uint4 gq[kPieces], bq[kPieces];
#pragma unroll
    for (int j = 0; j < kPieces; ++j) {
        gq[j] = __ldg(reinterpret_cast<const uint4*>(gamma) + sub + 8 * j);
        bq[j] = __ldg(reinterpret_cast<const uint4*>(beta) + sub + 8 * j);
    }
#pragma unroll 1
    for (int it = 0; it < 2; ++it) {
        const int row = warp * 8 + it * 4 + rsel;
        uint4* prow = reinterpret_cast<uint4*>(panel + row * stride);
        float v[kPieces][8];
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < kPieces; ++j) {
            unpack8(prow[sub + 8 * j], v[j]);
#pragma unroll
            for (int e = 0; e < 8; ++e) s += v[j][e];
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float mean = s * inv_d;
        float q = 0.f;
#pragma unroll
        for (int j = 0; j < kPieces; ++j)
#pragma unroll
            for (int e = 0; e < 8; ++e) { const float c = v[j][e] - mean; q = fmaf(c, c, q); }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
        const float rs = rsqrtf(q * inv_d + eps);
#pragma unroll
        for (int j = 0; j < kPieces; ++j) {
            float g[8], b[8], y[8];
            unpack8(gq[j], g);
            unpack8(bq[j], b);
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = fmaf((v[j][e] - mean) * rs, g[e], b[e]);
            const uint4 out = pack8(y);
            prow[sub + 8 * j] = out;
            if (write) *(reinterpret_cast<uint4*>(h + static_cast<size_t>(m0 + row) * d) + sub + 8 * j) = out;
        }
        if (write && sub == 0) { mu[m0 + row] = mean; rstd[m0 + row] = rs; }
    }
}

// ---------------------------------------------------------------- column sums (bias gradients, dgamma / dbeta)
// One unit: 32 columns (4 pieces of 16 bytes) x 64 row lanes, eight rows of a lane in flight (512
// rows are one trip to L2); the lanes' sums are added in lane order.  With xhat_of != nullptr it
// returns sum(in * xhat) in out0 and sum(in) in out1 (xhat = (xhat_of - mu) * rstd), else sum(in) in
// out0.  red: 2 x 64 x 32 floats.
__device__ __noinline__ void colsum_unit(const uint16_t* in, size_t ld, int T, int col0, const uint16_t* xhat_of, const float* mu,
                                         const float* rstd, float* out0, float* out1, int accumulate, float* red)
{
    const int tid = threadIdx.x, g = tid & 3, rl = tid >> 2;
    float s0[8], s1[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { s0[e] = 0.f; s1[e] = 0.f; }
    for (int r0 = rl; r0 < T; r0 += 64 * 8) {
        uint4 a[8], b[8];
        float m[8], rs[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int row = r0 + 64 * i;
            if (row < T) {
                a[i] = __ldcg(reinterpret_cast<const uint4*>(in + row * ld + col0) + g);
                if (xhat_of) {
                    b[i] = __ldcg(reinterpret_cast<const uint4*>(xhat_of + row * ld + col0) + g);
                    m[i] = __ldcg(mu + row);
                    rs[i] = __ldcg(rstd + row);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (r0 + 64 * i < T) {
                float v[8];
                unpack8(a[i], v);
                if (xhat_of) {
                    float xv[8];
                    unpack8(b[i], xv);
#pragma unroll
                    for (int e = 0; e < 8; ++e) { s0[e] = fmaf(v[e], (xv[e] - m[i]) * rs[i], s0[e]); s1[e] += v[e]; }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) s0[e] += v[e];
                }
            }
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) { red[rl * 32 + g * 8 + e] = s0[e]; red[2048 + rl * 32 + g * 8 + e] = s1[e]; }
    __syncthreads();
    if (tid < 32) {
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int l = 0; l < 64; ++l) { a0 += red[l * 32 + tid]; a1 += red[2048 + l * 32 + tid]; }
        out0[col0 + tid] = accumulate ? out0[col0 + tid] + a0 : a0;
        if (xhat_of) out1[col0 + tid] = accumulate ? out1[col0 + tid] + a1 : a1;
    }
    __syncthreads();
}

// ---------------------------------------------------------------- LayerNorm backward, one row per warp
// dx = resid + rstd * (g - mean(g) - xhat * mean(g * xhat)),  g = dh * gamma
template <int NP>
__device__ __forceinline__ void ln_bwd_row(const uint16_t* dh, const uint16_t* x, const float* mu, const float* rstd,
                                           const uint16_t* gamma, const uint16_t* resid, uint16_t* dx, int row)
{
    constexpr int d = 256 * NP;
    const int lane = threadIdx.x & 31;
    const float inv_d = 1.0f / d;
    uint4 qa[NP], qb[NP], qc[NP], qr[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        qa[i] = __ldcg(reinterpret_cast<const uint4*>(dh + static_cast<size_t>(row) * d) + lane + 32 * i);
        qb[i] = __ldcg(reinterpret_cast<const uint4*>(x + static_cast<size_t>(row) * d) + lane + 32 * i);
        qr[i] = __ldcg(reinterpret_cast<const uint4*>(resid + static_cast<size_t>(row) * d) + lane + 32 * i);
        qc[i] = __ldg(reinterpret_cast<const uint4*>(gamma) + lane + 32 * i);
    }
    const float m = __ldcg(mu + row), rs = __ldcg(rstd + row);
    float g[NP][8], xh[NP][8];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        float a[8], b[8], c[8];
        unpack8(qa[i], a);
        unpack8(qb[i], b);
        unpack8(qc[i], c);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            g[i][e] = a[e] * c[e];
            xh[i][e] = (b[e] - m) * rs;
            s1 += g[i][e];
            s2 = fmaf(g[i][e], xh[i][e], s2);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    s1 *= inv_d; s2 *= inv_d;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        float r[8], y[8];
        unpack8(qr[i], r);
#pragma unroll
        for (int e = 0; e < 8; ++e) y[e] = r[e] + rs * (g[i][e] - s1 - xh[i][e] * s2);
        *(reinterpret_cast<uint4*>(dx + static_cast<size_t>(row) * d) + lane + 32 * i) = pack8(y);
    }
}

// ---------------------------------------------------------------- attention units (head_dim 64)
// rowsum(dO * O) of one row of one head: 64 products added in column order.
__device__ __forceinline__ float delta_row(const uint16_t* dout, const uint16_t* o, size_t idx)
{
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float a[8], b[8];
        unpack8(__ldcg(reinterpret_cast<const uint4*>(dout + idx) + i), a);
        unpack8(__ldcg(reinterpret_cast<const uint4*>(o + idx) + i), b);
#pragma unroll
        for (int e = 0; e < 8; ++e) s = fmaf(a[e], b[e], s);
    }
    return s;
}

// Forward: 64 query rows of one head.  Warps w and w + 4 share rows 16 (w % 4) .. + 15; each takes one
// half (32 keys) of every 64-key block and runs its own online softmax over its keys, with scores and P
// in registers; the two partial results (running maximum, sum, unnormalised O) are merged at the end
// through shared memory.  `mrg` is 4 x (16 x 64 + 32) floats.
__device__ __noinline__ void attn_fwd_unit(const WholeLayerArgs& p, int b, int h, int qb, uint32_t sm, float* mrg)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, rw = warp & 3, kh = warp >> 2;
    const size_t ld = 3 * static_cast<size_t>(p.d);
    const uint16_t* qkv = static_cast<const uint16_t*>(p.qkv);
    const uint16_t* base = qkv + static_cast<size_t>(b) * p.S * ld + h * 64;
    const uint32_t sQ = sm;                                 // K / V of block j in chunks 1 + 2 (j & 1), 2 + 2 (j & 1)
    const float sl2 = p.scale * 1.4426950408889634f;
    auto load_kv = [&](int j) {
        stage_chunk(sm + (1 + 2 * (j & 1)) * kChunk, base + static_cast<size_t>(j) * 64 * ld + p.d, ld, tid);
        stage_chunk(sm + (2 + 2 * (j & 1)) * kChunk, base + static_cast<size_t>(j) * 64 * ld + 2 * p.d, ld, tid);
    };
    stage_chunk(sQ, base + static_cast<size_t>(qb) * 64 * ld, ld, tid);
    load_kv(0);
    cp_async_commit();
    float oacc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) oacc[i][e] = 0.f;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    for (int j = 0; j <= qb; ++j) {
        if (j < qb) load_kv(j + 1);                         // the next block travels while this one is used
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t sK = sm + (1 + 2 * (j & 1)) * kChunk, sV = sK + kChunk;
        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[i][e] = 0.f;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            uint32_t qf[4];
            frag_a_k(sQ, rw * 16, kk, lane, qf);
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                uint32_t bf[4];
                frag_b_k(sK, kh * 32 + np * 16, kk, lane, bf);
                mma16816(s[2 * np], qf, bf[0], bf[1]);
                mma16816(s[2 * np + 1], qf, bf[2], bf[3]);
            }
        }
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float t = s[ni][e] * sl2;
                if (j == qb) {
                    const int key = kh * 32 + ni * 8 + 2 * (lane & 3) + (e & 1), row = rw * 16 + (lane >> 2) + 8 * (e >> 1);
                    if (key > row) t = -INFINITY;
                }
                s[ni][e] = t;
                mx[e >> 1] = fmaxf(mx[e >> 1], t);
            }
        float alpha[2], mb[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
            mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
            const float mn = fmaxf(m[hh], mx[hh]);
            mb[hh] = mn == -INFINITY ? 0.f : mn;            // a half may see only masked keys of a row
            alpha[hh] = exp2f(m[hh] - mb[hh]);
            m[hh] = mn;
            l[hh] *= alpha[hh];
        }
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float pe = exp2f(s[ni][e] - mb[e >> 1]);
                s[ni][e] = pe;
                l[e >> 1] += pe;
            }
#pragma unroll
        for (int ni = 0; ni < 8; ++ni)
#pragma unroll
            for (int e = 0; e < 4; ++e) oacc[ni][e] *= alpha[e >> 1];
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            uint32_t a[4] = {pack_bf16(s[2 * kk][0], s[2 * kk][1]), pack_bf16(s[2 * kk][2], s[2 * kk][3]),
                             pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]), pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3])};
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t bf[4];
                frag_b_mn(sV, np * 16, kh * 2 + kk, lane, bf);
                mma16816(oacc[2 * np], a, bf[0], bf[1]);
                mma16816(oacc[2 * np + 1], a, bf[2], bf[3]);
            }
        }
        __syncthreads();                                    // K and V may be overwritten
    }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 1);
        l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 2);
    }
    // merge: the upper half hands (m, l, O) to the lower half
    float* mine = mrg + rw * (16 * 64 + 32);
    if (kh == 1) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = (lane >> 2) + 8 * hh;
#pragma unroll
            for (int ni = 0; ni < 8; ++ni)
                *reinterpret_cast<float2*>(mine + r * 64 + ni * 8 + 2 * (lane & 3)) = make_float2(oacc[ni][2 * hh], oacc[ni][2 * hh + 1]);
            if ((lane & 3) == 0) { mine[1024 + r] = m[hh]; mine[1040 + r] = l[hh]; }
        }
    }
    __syncthreads();
    if (kh == 0) {
        uint16_t* o = static_cast<uint16_t*>(p.o);
        float* lse = static_cast<float*>(p.lse);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = (lane >> 2) + 8 * hh;
            const float m2 = mine[1024 + r], l2 = mine[1040 + r];
            const float mt = fmaxf(m[hh], m2);              // the lower half always sees key 0: finite
            const float c1 = exp2f(m[hh] - mt), c2 = m2 == -INFINITY ? 0.f : exp2f(m2 - mt);
            const float lt = l[hh] * c1 + l2 * c2, inv = 1.0f / lt;
            const int q = qb * 64 + rw * 16 + r;
            const size_t row = static_cast<size_t>(b) * p.S + q;
#pragma unroll
            for (int ni = 0; ni < 8; ++ni) {
                const float2 o2 = *reinterpret_cast<const float2*>(mine + r * 64 + ni * 8 + 2 * (lane & 3));
                store_bf16x2(o, row * p.d + h * 64 + ni * 8 + 2 * (lane & 3), (oacc[ni][2 * hh] * c1 + o2.x * c2) * inv,
                             (oacc[ni][2 * hh + 1] * c1 + o2.y * c2) * inv);
            }
            if ((lane & 3) == 0) lse[(static_cast<size_t>(b) * p.H + h) * p.S + q] = mt * 0.6931471805599453f + logf(lt);
        }
    }
    __syncthreads();                                        // the merge area may be rewritten by the next unit
}

// Backward, dQ of 64 query rows of one head: per key block S and dP are rebuilt, dS = P (dP - delta)
// goes straight from the accumulator registers into the A operand of dQ += dS K.  Warps w and w + 4
// share rows 16 (w % 4) .. + 15 and split every key block in halves; the two partial dQ are added (lower
// half first) through shared memory.  `mrg` is 4 x 16 x 64 floats.
__device__ __noinline__ void attn_dq_unit(const WholeLayerArgs& p, int b, int h, int qb, uint32_t sm, float* vec, float* mrg)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, rw = warp & 3, kh = warp >> 2;
    const size_t ld = 3 * static_cast<size_t>(p.d);
    const uint16_t* base = static_cast<const uint16_t*>(p.qkv) + static_cast<size_t>(b) * p.S * ld + h * 64;
    const uint16_t* dout = static_cast<const uint16_t*>(p.td0);
    const uint16_t* o = static_cast<const uint16_t*>(p.o);
    const uint32_t sQ = sm, sDO = sm + kChunk;              // K / V of block j in chunks 2 + 2 (j & 1), 3 + 2 (j & 1)
    const float sl2 = p.scale * 1.4426950408889634f;
    const size_t row0 = static_cast<size_t>(b) * p.S + qb * 64;
    auto load_kv = [&](int j) {
        stage_chunk(sm + (2 + 2 * (j & 1)) * kChunk, base + static_cast<size_t>(j) * 64 * ld + p.d, ld, tid);
        stage_chunk(sm + (3 + 2 * (j & 1)) * kChunk, base + static_cast<size_t>(j) * 64 * ld + 2 * p.d, ld, tid);
    };
    stage_chunk(sQ, base + static_cast<size_t>(qb) * 64 * ld, ld, tid);
    stage_chunk(sDO, dout + row0 * p.d + h * 64, p.d, tid);
    load_kv(0);
    cp_async_commit();
    if (tid < 64) vec[tid] = delta_row(dout, o, (row0 + tid) * p.d + h * 64);
    float lse2[2], dlt[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
        lse2[hh] = __ldcg(static_cast<const float*>(p.lse) + (static_cast<size_t>(b) * p.H + h) * p.S + qb * 64 + rw * 16 + (lane >> 2) + 8 * hh) * 1.4426950408889634f;
    float dq[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) dq[i][e] = 0.f;
    for (int j = 0; j <= qb; ++j) {
        if (j < qb) load_kv(j + 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t sK = sm + (2 + 2 * (j & 1)) * kChunk, sV = sK + kChunk;
        if (j == 0) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) dlt[hh] = vec[rw * 16 + (lane >> 2) + 8 * hh];
        }
        float s[4][4], dp[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) { s[i][e] = 0.f; dp[i][e] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            uint32_t qf[4], dof[4];
            frag_a_k(sQ, rw * 16, kk, lane, qf);
            frag_a_k(sDO, rw * 16, kk, lane, dof);
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                uint32_t bf[4];
                frag_b_k(sK, kh * 32 + np * 16, kk, lane, bf);
                mma16816(s[2 * np], qf, bf[0], bf[1]);
                mma16816(s[2 * np + 1], qf, bf[2], bf[3]);
                frag_b_k(sV, kh * 32 + np * 16, kk, lane, bf);
                mma16816(dp[2 * np], dof, bf[0], bf[1]);
                mma16816(dp[2 * np + 1], dof, bf[2], bf[3]);
            }
        }
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float pe = exp2f(fmaf(s[ni][e], sl2, -lse2[e >> 1]));
                if (j == qb) {
                    const int key = kh * 32 + ni * 8 + 2 * (lane & 3) + (e & 1), row = rw * 16 + (lane >> 2) + 8 * (e >> 1);
                    if (key > row) pe = 0.f;
                }
                s[ni][e] = pe * (dp[ni][e] - dlt[e >> 1]);
            }
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            uint32_t a[4] = {pack_bf16(s[2 * kk][0], s[2 * kk][1]), pack_bf16(s[2 * kk][2], s[2 * kk][3]),
                             pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]), pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3])};
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t bf[4];
                frag_b_mn(sK, np * 16, kh * 2 + kk, lane, bf);
                mma16816(dq[2 * np], a, bf[0], bf[1]);
                mma16816(dq[2 * np + 1], a, bf[2], bf[3]);
            }
        }
        __syncthreads();
    }
    float* mine = mrg + rw * (16 * 64);
    if (kh == 1) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
            for (int ni = 0; ni < 8; ++ni)
                *reinterpret_cast<float2*>(mine + ((lane >> 2) + 8 * hh) * 64 + ni * 8 + 2 * (lane & 3)) = make_float2(dq[ni][2 * hh], dq[ni][2 * hh + 1]);
    }
    __syncthreads();
    if (kh == 0) {
        uint16_t* dqkv = static_cast<uint16_t*>(p.big);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = (lane >> 2) + 8 * hh;
            const size_t row = row0 + rw * 16 + r;
#pragma unroll
            for (int ni = 0; ni < 8; ++ni) {
                const float2 o2 = *reinterpret_cast<const float2*>(mine + r * 64 + ni * 8 + 2 * (lane & 3));
                store_bf16x2(dqkv, row * ld + h * 64 + ni * 8 + 2 * (lane & 3), (dq[ni][2 * hh] + o2.x) * p.scale,
                             (dq[ni][2 * hh + 1] + o2.y) * p.scale);
            }
        }
    }
    __syncthreads();
}

// Backward, dK and dV of 64 key rows of one head: per query block the transposed scores K Q^T and
// V dO^T are built, so that P^T and dS^T come out of the accumulators as A operands.  Warps w and w + 4
// share keys 16 (w % 4) .. + 15 and split every query block in halves; the partial dK and dV are added
// (lower half first) through shared memory.  `mrg` is 2 x 4 x 16 x 64 floats.
__device__ __noinline__ void attn_dkdv_unit(const WholeLayerArgs& p, int b, int h, int kb, uint32_t sm, float* vec, float* mrg)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, rw = warp & 3, qh = warp >> 2;
    const size_t ld = 3 * static_cast<size_t>(p.d);
    const uint16_t* base = static_cast<const uint16_t*>(p.qkv) + static_cast<size_t>(b) * p.S * ld + h * 64;
    const uint16_t* dout = static_cast<const uint16_t*>(p.td0);
    const uint16_t* o = static_cast<const uint16_t*>(p.o);
    const uint32_t sK = sm, sV = sm + kChunk;               // Q / dO of block i in chunks 2 + 2 (i & 1), 3 + 2 (i & 1)
    const float sl2 = p.scale * 1.4426950408889634f;
    const size_t seq0 = static_cast<size_t>(b) * p.S;
    float* v_lse = vec;                                     // [S] lse * log2(e)
    float* v_dlt = vec + kMaxS;                             // [S]
    auto load_q = [&](int i) {
        stage_chunk(sm + (2 + 2 * (i & 1)) * kChunk, base + static_cast<size_t>(i) * 64 * ld, ld, tid);
        stage_chunk(sm + (3 + 2 * (i & 1)) * kChunk, dout + (seq0 + i * 64) * p.d + h * 64, p.d, tid);
    };
    stage_chunk(sK, base + static_cast<size_t>(kb) * 64 * ld + p.d, ld, tid);
    stage_chunk(sV, base + static_cast<size_t>(kb) * 64 * ld + 2 * p.d, ld, tid);
    load_q(kb);
    cp_async_commit();
    for (int r = kb * 64 + tid; r < p.S; r += kThreads) {
        v_lse[r] = __ldcg(static_cast<const float*>(p.lse) + (static_cast<size_t>(b) * p.H + h) * p.S + r) * 1.4426950408889634f;
        v_dlt[r] = delta_row(dout, o, (seq0 + r) * p.d + h * 64);
    }
    float dk[8][4], dv[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) { dk[i][e] = 0.f; dv[i][e] = 0.f; }
    const int nqb = p.S >> 6;
    for (int i = kb; i < nqb; ++i) {
        if (i + 1 < nqb) load_q(i + 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t sQ = sm + (2 + 2 * (i & 1)) * kChunk, sDO = sQ + kChunk;
        float st[4][4], dpt[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int e = 0; e < 4; ++e) { st[a][e] = 0.f; dpt[a][e] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            uint32_t kf[4], vf[4];
            frag_a_k(sK, rw * 16, kk, lane, kf);
            frag_a_k(sV, rw * 16, kk, lane, vf);
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                uint32_t bf[4];
                frag_b_k(sQ, qh * 32 + np * 16, kk, lane, bf);
                mma16816(st[2 * np], kf, bf[0], bf[1]);
                mma16816(st[2 * np + 1], kf, bf[2], bf[3]);
                frag_b_k(sDO, qh * 32 + np * 16, kk, lane, bf);
                mma16816(dpt[2 * np], vf, bf[0], bf[1]);
                mma16816(dpt[2 * np + 1], vf, bf[2], bf[3]);
            }
        }
        // st -> P^T (kept for dV), dpt -> dS^T
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int qcol = qh * 32 + ni * 8 + 2 * (lane & 3) + (e & 1), q = i * 64 + qcol;
                float pe = exp2f(fmaf(st[ni][e], sl2, -v_lse[q]));
                if (i == kb) {
                    const int key = rw * 16 + (lane >> 2) + 8 * (e >> 1);
                    if (key > qcol) pe = 0.f;
                }
                st[ni][e] = pe;
                dpt[ni][e] = pe * (dpt[ni][e] - v_dlt[q]);
            }
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            uint32_t a[4] = {pack_bf16(st[2 * kk][0], st[2 * kk][1]), pack_bf16(st[2 * kk][2], st[2 * kk][3]),
                             pack_bf16(st[2 * kk + 1][0], st[2 * kk + 1][1]), pack_bf16(st[2 * kk + 1][2], st[2 * kk + 1][3])};
            uint32_t c[4] = {pack_bf16(dpt[2 * kk][0], dpt[2 * kk][1]), pack_bf16(dpt[2 * kk][2], dpt[2 * kk][3]),
                             pack_bf16(dpt[2 * kk + 1][0], dpt[2 * kk + 1][1]), pack_bf16(dpt[2 * kk + 1][2], dpt[2 * kk + 1][3])};
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t bf[4];
                frag_b_mn(sDO, np * 16, qh * 2 + kk, lane, bf);
                mma16816(dv[2 * np], a, bf[0], bf[1]);
                mma16816(dv[2 * np + 1], a, bf[2], bf[3]);
                frag_b_mn(sQ, np * 16, qh * 2 + kk, lane, bf);
                mma16816(dk[2 * np], c, bf[0], bf[1]);
                mma16816(dk[2 * np + 1], c, bf[2], bf[3]);
            }
        }
        __syncthreads();
    }
    float* mk = mrg + rw * (16 * 64);
    float* mv = mrg + 4 * 16 * 64 + rw * (16 * 64);
    if (qh == 1) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
            for (int ni = 0; ni < 8; ++ni) {
                const int at = ((lane >> 2) + 8 * hh) * 64 + ni * 8 + 2 * (lane & 3);
                *reinterpret_cast<float2*>(mk + at) = make_float2(dk[ni][2 * hh], dk[ni][2 * hh + 1]);
                *reinterpret_cast<float2*>(mv + at) = make_float2(dv[ni][2 * hh], dv[ni][2 * hh + 1]);
            }
    }
    __syncthreads();
    if (qh == 0) {
        uint16_t* dqkv = static_cast<uint16_t*>(p.big);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = (lane >> 2) + 8 * hh;
            const size_t row = seq0 + kb * 64 + rw * 16 + r;
#pragma unroll
            for (int ni = 0; ni < 8; ++ni) {
                const int at = r * 64 + ni * 8 + 2 * (lane & 3);
                const float2 k2 = *reinterpret_cast<const float2*>(mk + at), v2 = *reinterpret_cast<const float2*>(mv + at);
                const size_t dst = row * ld + h * 64 + ni * 8 + 2 * (lane & 3);
                store_bf16x2(dqkv, dst + p.d, (dk[ni][2 * hh] + k2.x) * p.scale, (dk[ni][2 * hh + 1] + k2.y) * p.scale);
                store_bf16x2(dqkv, dst + 2 * p.d, dv[ni][2 * hh] + v2.x, dv[ni][2 * hh + 1] + v2.y);
            }
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------- the phases
struct Ctx {
    const WholeLayerArgs& p;
    uint8_t* smem;
    uint32_t sm;                // shared-memory address of smem
    int* flag;
    unsigned* sem;
    float* ws;
};

// The accumulators leave the registers through a 64 x 64 fp32 tile in shared memory; the epilogue is
// then a rolled loop over 16-byte pieces of the output (8 columns of a row per thread and turn), short
// enough to stay in the instruction cache and storing whole 16-byte pieces.
__device__ __forceinline__ void acc_to_smem(const float (&acc)[2][2][4], float* tile)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = (warp & 1) * 32 + (lane >> 2), c = (warp >> 1) * 16 + 2 * (lane & 3);
#pragma unroll
    for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int ni = 0; ni < 2; ++ni)
#pragma unroll
            for (int h = 0; h < 2; ++h)
                *reinterpret_cast<float2*>(tile + (r + mi * 16 + h * 8) * kAccStride + c + ni * 8) =
                    make_float2(acc[mi][ni][2 * h], acc[mi][ni][2 * h + 1]);
    __syncthreads();
}
__device__ __forceinline__ void tile_piece(const float* tile, int row, int c8, float (&v)[8])
{
    const float4 a = *reinterpret_cast<const float4*>(tile + row * kAccStride + c8);
    const float4 b = *reinterpret_cast<const float4*>(tile + row * kAccStride + c8 + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// Forward GEMM tile with bias and one of: nothing, residual, GeLU (writes u and a).  The operand
// chunks and the residual tile are requested first; LayerNorm (LN) runs while the weights travel.
enum { kFwdBias = 0, kFwdResid = 1, kFwdGelu = 2 };
template <bool LN>
__device__ __noinline__ void fwd_gemm_unit(const Ctx& c, int u, int mode, const uint16_t* A, int K, const uint16_t* W,
                                           const uint16_t* bias, int N, int nslices, const uint16_t* resid, uint16_t* out,
                                           uint16_t* out_act, const uint16_t* ln_g, const uint16_t* ln_b, uint16_t* ln_h,
                                           float* ln_mu, float* ln_rs)
{
    const WholeLayerArgs& p = c.p;
    const int tile = u / nslices, slice = u % nslices, ntn = N >> 6, tm = tile / ntn, tn = tile % ntn;
    const int m0 = tm * 64, n0 = tn * 64, kper = K / nslices, tid = threadIdx.x;
    float acc[2][2][4];
    const TileGemm<false, false, LN> g{A, static_cast<size_t>(K), W, static_cast<size_t>(K), m0, n0, LN ? 0 : slice * kper,
                                       (LN ? K : kper) >> 6, c.sm + kSmStage};
    const int stride = (p.d + 8) * 2;
    if (LN) {
        ln_stage_rows(A, p.d, m0, c.sm + kSmPanel, stride);
        cp_async_commit();
    }
    if (mode == kFwdResid) stage_chunk(c.sm + kSmAux, resid + static_cast<size_t>(m0) * N + n0, N, tid);   // rides with the first chunk
    g.prefetch();
    if (LN) {
        cp_async_wait<kStages - 1>();                       // the rows of x have landed (the weight chunks may not have)
        __syncthreads();
        if (p.d == 256) ln_rows_in_panel<1>(ln_g, ln_b, p.eps, m0, c.smem + kSmPanel, stride, tn == 0, ln_h, ln_mu, ln_rs);
        else ln_rows_in_panel<2>(ln_g, ln_b, p.eps, m0, c.smem + kSmPanel, stride, tn == 0, ln_h, ln_mu, ln_rs);
        g.run(acc, c.sm + kSmPanel, stride);
    } else {
        g.run(acc, 0, 0);
        if (!splitk_combine(acc, c.ws, c.sem, tile, slice, nslices, c.flag)) return;
    }
    float* tl = reinterpret_cast<float*>(c.smem + kSmAcc);
    acc_to_smem(acc, tl);
    const int act = p.act, c8 = (tid & 7) * 8;
    float bv[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(bias + n0 + c8)), bv);
#pragma unroll 1
    for (int it = 0; it < 2; ++it) {
        const int row = (tid >> 3) + it * 32;
        float v[8];
        tile_piece(tl, row, c8, v);
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] += bv[e];
        if (mode == kFwdResid) {
            float r[8];
            unpack8(*reinterpret_cast<const uint4*>(c.smem + kSmAux + swz(row, tid & 7)), r);
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] += r[e];
        }
        const size_t idx = static_cast<size_t>(m0 + row) * N + n0 + c8;
        *reinterpret_cast<uint4*>(out + idx) = pack8(v);
        if (mode == kFwdGelu) {
#pragma unroll
            for (int e = 0; e < 8; e += 2) gelu2(v[e], v[e + 1], act);
            *reinterpret_cast<uint4*>(out_act + idx) = pack8(v);
        }
    }
    __syncthreads();                                        // the accumulator tile and the aux chunk may be rewritten
}

// Data-gradient tile: out[T, N] = A[T, K] W[K, N] (W stored [K][N]); with u != nullptr the result is
// multiplied by GeLU'(u).
__device__ __noinline__ void dgrad_unit(const Ctx& c, int u, const uint16_t* A, int K, const uint16_t* W, int N, int nslices,
                                        const uint16_t* gelu_u, uint16_t* out)
{
    const int tile = u / nslices, slice = u % nslices, ntn = N >> 6, m0 = (tile / ntn) * 64, n0 = (tile % ntn) * 64;
    const int kper = K / nslices, tid = threadIdx.x;
    float acc[2][2][4];
    const TileGemm<false, true, false> g{A, static_cast<size_t>(K), W, static_cast<size_t>(N), m0, n0, slice * kper, kper >> 6,
                                         c.sm + kSmStage};
    if (gelu_u) stage_chunk(c.sm + kSmAux, gelu_u + static_cast<size_t>(m0) * N + n0, N, tid);
    g.prefetch();
    g.run(acc, 0, 0);
    if (!splitk_combine(acc, c.ws, c.sem, tile, slice, nslices, c.flag)) return;
    float* tl = reinterpret_cast<float*>(c.smem + kSmAcc);
    acc_to_smem(acc, tl);
    const int act = c.p.act, c8 = (tid & 7) * 8;
#pragma unroll 1
    for (int it = 0; it < 2; ++it) {
        const int row = (tid >> 3) + it * 32;
        float v[8];
        tile_piece(tl, row, c8, v);
        if (gelu_u) {
            float uv[8];
            unpack8(*reinterpret_cast<const uint4*>(c.smem + kSmAux + swz(row, tid & 7)), uv);
#pragma unroll
            for (int e = 0; e < 8; e += 2) gelu_grad_mul2(v[e], v[e + 1], uv[e], uv[e + 1], act);
        }
        *reinterpret_cast<uint4*>(out + static_cast<size_t>(m0 + row) * N + n0 + c8) = pack8(v);
    }
    __syncthreads();
}

// Weight-gradient tile: dW[M, N] (+)= A[T, M]^T B[T, N], fp32.
__device__ __noinline__ void wgrad_unit(const Ctx& c, int u, const uint16_t* A, int M, const uint16_t* B, int N, float* dW)
{
    const int ntn = N >> 6, m0 = (u / ntn) * 64, n0 = (u % ntn) * 64, tid = threadIdx.x;
    float acc[2][2][4];
    const TileGemm<true, true, false> g{A, static_cast<size_t>(M), B, static_cast<size_t>(N), m0, n0, 0, c.p.T >> 6, c.sm + kSmStage};
    g.prefetch();
    float4 old[4];
    const int c4 = (tid & 15) * 4;
    if (c.p.accumulate) {
#pragma unroll
        for (int it = 0; it < 4; ++it) old[it] = *reinterpret_cast<const float4*>(dW + static_cast<size_t>(m0 + (tid >> 4) + it * 16) * N + n0 + c4);
    }
    g.run(acc, 0, 0);
    float* tl = reinterpret_cast<float*>(c.smem + kSmAcc);
    acc_to_smem(acc, tl);
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int row = (tid >> 4) + it * 16;
        float4 v = *reinterpret_cast<const float4*>(tl + row * kAccStride + c4);
        if (c.p.accumulate) { v.x += old[it].x; v.y += old[it].y; v.z += old[it].z; v.w += old[it].w; }
        *reinterpret_cast<float4*>(dW + static_cast<size_t>(m0 + row) * N + n0 + c4) = v;
    }
    __syncthreads();
}

__device__ __forceinline__ const uint16_t* cu16(const void* q) { return static_cast<const uint16_t*>(q); }
__device__ __forceinline__ uint16_t* u16(void* q) { return static_cast<uint16_t*>(q); }
__device__ __forceinline__ float* f32(void* q) { return static_cast<float*>(q); }

__global__ void __launch_bounds__(kThreads, 1) whole_layer_fwd_kernel(const __grid_constant__ WholeLayerArgs p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const Ctx c{p, smem, smem_u32(smem), reinterpret_cast<int*>(smem + kSmFlag), p.sync + 2, f32(p.splitk)};
    if (*reinterpret_cast<volatile int*>(&p.status->code) != 0) return;
    const int T = p.T, d = p.d, F = p.F, G = gridDim.x, tm = T >> 6;
    // 1: qkv = LN1(x) Wqkv^T + bqkv (h1, mean, rstd written by the first column tile of each row block)
    for (int u = blockIdx.x; u < tm * (3 * d >> 6); u += G)
        fwd_gemm_unit<true>(c, u, kFwdBias, cu16(p.x), d, cu16(p.w_qkv), cu16(p.b_qkv), 3 * d, 1, nullptr, u16(p.qkv), nullptr,
                            cu16(p.ln1_g), cu16(p.ln1_b), u16(p.h1), f32(p.mu1), f32(p.r1));
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 2: o = attention(qkv)
    {
        const int nqb = p.S >> 6, n = p.B * p.H * nqb;
        for (int u = blockIdx.x; u < n; u += G) {
            const int qb = nqb - 1 - u / (p.B * p.H), bh = u % (p.B * p.H);      // long rows first
            attn_fwd_unit(p, bh / p.H, bh % p.H, qb, c.sm + kSmStage, reinterpret_cast<float*>(smem + kSmPanel));
        }
    }
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 3: x1 = x + o Wo^T + bo
    for (int u = blockIdx.x; u < tm * (d >> 6) * p.split_o; u += G)
        fwd_gemm_unit<false>(c, u, kFwdResid, cu16(p.o), d, cu16(p.w_o), cu16(p.b_o), d, p.split_o, cu16(p.x), u16(p.x1), nullptr,
                             nullptr, nullptr, nullptr, nullptr, nullptr);
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 4: u = LN2(x1) W1^T + b1, a = GeLU(u)
    for (int u = blockIdx.x; u < tm * (F >> 6); u += G)
        fwd_gemm_unit<true>(c, u, kFwdGelu, cu16(p.x1), d, cu16(p.w_fc1), cu16(p.b_fc1), F, 1, nullptr, u16(p.u), u16(p.a),
                            cu16(p.ln2_g), cu16(p.ln2_b), u16(p.h2), f32(p.mu2), f32(p.r2));
    if (!p.with_fc2) return;
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 5: y = x1 + a W2^T + b2
    for (int u = blockIdx.x; u < tm * (d >> 6) * p.split_fc2; u += G)
        fwd_gemm_unit<false>(c, u, kFwdResid, cu16(p.a), F, cu16(p.w_fc2), cu16(p.b_fc2), d, p.split_fc2, cu16(p.x1), u16(p.y), nullptr,
                             nullptr, nullptr, nullptr, nullptr, nullptr);
}

__global__ void __launch_bounds__(kThreads, 1) whole_layer_bwd_kernel(const __grid_constant__ WholeLayerArgs p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const Ctx c{p, smem, smem_u32(smem), reinterpret_cast<int*>(smem + kSmFlag), p.sync + 2, f32(p.splitk)};
    if (*reinterpret_cast<volatile int*>(&p.status->code) != 0) return;
    const int T = p.T, d = p.d, F = p.F, G = gridDim.x, tm = T >> 6, warp = threadIdx.x >> 5;
    float* red = reinterpret_cast<float*>(smem + kSmPanel);
    float* vec = reinterpret_cast<float*>(smem + kSmVec);
    const int acc = p.accumulate;
    // 1: du = (dy W2) * GeLU'(u);  dW2 = dy^T a;  db2 = colsum(dy)
    {
        const int n0 = (d >> 6) * (F >> 6), n1 = n0 + tm * (F >> 6), n2 = n1 + (d >> 5);
        for (int u = blockIdx.x; u < n2; u += G) {
            if (u < n0) wgrad_unit(c, u, cu16(p.dy), d, cu16(p.a), F, f32(p.g_w_fc2));
            else if (u < n1) dgrad_unit(c, u - n0, cu16(p.dy), d, cu16(p.w_fc2), F, 1, cu16(p.u), u16(p.big));
            else colsum_unit(cu16(p.dy), d, T, (u - n1) * 32, nullptr, nullptr, nullptr, f32(p.g_b_fc2), nullptr, acc, red);
        }
    }
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 2: dh2 = du W1;  dW1 = du^T h2;  db1 = colsum(du)
    {
        const int n0 = (F >> 6) * (d >> 6), n1 = n0 + tm * (d >> 6) * p.split_dh2, n2 = n1 + (F >> 5);
        for (int u = blockIdx.x; u < n2; u += G) {
            if (u < n0) wgrad_unit(c, u, cu16(p.big), F, cu16(p.h2), d, f32(p.g_w_fc1));
            else if (u < n1) dgrad_unit(c, u - n0, cu16(p.big), F, cu16(p.w_fc1), d, p.split_dh2, nullptr, u16(p.td0));
            else colsum_unit(cu16(p.big), F, T, (u - n1) * 32, nullptr, nullptr, nullptr, f32(p.g_b_fc1), nullptr, acc, red);
        }
    }
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 3: dx1 = dy + LN2bwd(dh2) (a row per warp);  dgamma2, dbeta2
    {
        const int n0 = T >> 3, n1 = n0 + (d >> 5);
        for (int u = blockIdx.x; u < n1; u += G) {
            if (u < n0) {
                if (d == 256) ln_bwd_row<1>(cu16(p.td0), cu16(p.x1), f32(p.mu2), f32(p.r2), cu16(p.ln2_g), cu16(p.dy), u16(p.dx1), u * 8 + warp);
                else ln_bwd_row<2>(cu16(p.td0), cu16(p.x1), f32(p.mu2), f32(p.r2), cu16(p.ln2_g), cu16(p.dy), u16(p.dx1), u * 8 + warp);
            }
            else colsum_unit(cu16(p.td0), d, T, (u - n0) * 32, cu16(p.x1), f32(p.mu2), f32(p.r2), f32(p.g_ln2_g), f32(p.g_ln2_b), acc, red);
        }
    }
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 4: dout = dx1 Wo;  dWo = dx1^T o;  dbo = colsum(dx1)
    {
        const int n0 = (d >> 6) * (d >> 6), n1 = n0 + tm * (d >> 6) * p.split_o, n2 = n1 + (d >> 5);
        for (int u = blockIdx.x; u < n2; u += G) {
            if (u < n0) wgrad_unit(c, u, cu16(p.dx1), d, cu16(p.o), d, f32(p.g_w_o));
            else if (u < n1) dgrad_unit(c, u - n0, cu16(p.dx1), d, cu16(p.w_o), d, p.split_o, nullptr, u16(p.td0));
            else colsum_unit(cu16(p.dx1), d, T, (u - n1) * 32, nullptr, nullptr, nullptr, f32(p.g_b_o), nullptr, acc, red);
        }
    }
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 5: dqkv = attention backward (delta is taken by each unit from dout and o)
    {
        const int nb = p.S >> 6, BH = p.B * p.H, n = BH * nb;
        for (int u = blockIdx.x; u < 2 * n; u += G) {
            const int v = u >> 1, blk = v / BH, bh = v % BH;
            if (u & 1) attn_dq_unit(p, bh / p.H, bh % p.H, nb - 1 - blk, c.sm + kSmStage, vec, red);     // long rows first
            else attn_dkdv_unit(p, bh / p.H, bh % p.H, blk, c.sm + kSmStage, vec, red);                  // long columns first
            __syncthreads();
        }
    }
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 6: dh1 = dqkv Wqkv;  dWqkv = dqkv^T h1;  dbqkv = colsum(dqkv)
    {
        const int n0 = (3 * d >> 6) * (d >> 6), n1 = n0 + tm * (d >> 6) * p.split_dh1, n2 = n1 + (3 * d >> 5);
        for (int u = blockIdx.x; u < n2; u += G) {
            if (u < n0) wgrad_unit(c, u, cu16(p.big), 3 * d, cu16(p.h1), d, f32(p.g_w_qkv));
            else if (u < n1) dgrad_unit(c, u - n0, cu16(p.big), 3 * d, cu16(p.w_qkv), d, p.split_dh1, nullptr, u16(p.td0));
            else colsum_unit(cu16(p.big), 3 * d, T, (u - n1) * 32, nullptr, nullptr, nullptr, f32(p.g_b_qkv), nullptr, acc, red);
        }
    }
    if (!grid_barrier(p.sync, p.status, c.flag)) return;
    // 7: dx = dx1 + LN1bwd(dh1);  dgamma1, dbeta1
    {
        const int n0 = T >> 3, n1 = n0 + (d >> 5);
        for (int u = blockIdx.x; u < n1; u += G) {
            if (u < n0) {
                if (d == 256) ln_bwd_row<1>(cu16(p.td0), cu16(p.x), f32(p.mu1), f32(p.r1), cu16(p.ln1_g), cu16(p.dx1), u16(p.dx), u * 8 + warp);
                else ln_bwd_row<2>(cu16(p.td0), cu16(p.x), f32(p.mu1), f32(p.r1), cu16(p.ln1_g), cu16(p.dx1), u16(p.dx), u * 8 + warp);
            }
            else colsum_unit(cu16(p.td0), d, T, (u - n0) * 32, cu16(p.x), f32(p.mu1), f32(p.r1), f32(p.g_ln1_g), f32(p.g_ln1_b), acc, red);
        }
    }
}

cudaError_t launch_coop(void (*kern)(const WholeLayerArgs), int grid, cudaStream_t st, const WholeLayerArgs& a)
{
    Tuning& tn = tuning();
    if (tn.fail_launch_countdown > 0 && --tn.fail_launch_countdown == 0) return cudaErrorLaunchFailure;   // injected by a test
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmBytes; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, a);
}

}  // namespace

const char* configure_whole_layer()
{
    if (cudaFuncSetAttribute(whole_layer_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmBytes) != cudaSuccess ||
        cudaFuncSetAttribute(whole_layer_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmBytes) != cudaSuccess)
        return "could not set the whole-layer kernels' shared-memory size";
    return nullptr;
}

const char* whole_layer_unsupported(int T, int d, int H, int dh, int F, int S)
{
    (void)H;
    if (dh != 64) return "the whole-layer kernel needs head_dim 64";
    if (d > kMaxD) return "the whole-layer kernel needs d_model <= 512";
    if (S > kMaxS) return "the whole-layer kernel needs seq_len <= 1024";
    if ((T >> 6) * (d >> 6) > kWholeLayerMaxTiles) return "the whole-layer kernel needs (tokens / 64) * (d_model / 64) <= 1024";
    if (F % 64 != 0 || d % 256 != 0 || T % 64 != 0) return "the whole-layer kernel needs tokens and d_ff in multiples of 64";
    return nullptr;
}

// Slices of the K range of a GEMM with `tiles` output tiles.  Meeting the other slices costs three
// trips to L2 (partial tile out, ticket, partial tiles back in), about as much as eight 64-wide
// blocks of products, so only long K ranges are cut: into as many slices as keep every slice at
// least two blocks long, divide the block count, and fit into `room` CTAs - what one round of the grid
// has left beside the other GEMM of the phase (the short column-sum units go to a second round).
static int pick_slices(int tiles, int K, int room)
{
    const int grid = room;
    const int blocks = K / 64;
    int best = 1;
    if (blocks < 12) return 1;
    for (int s = 2; s <= 8; ++s)
        if (blocks % s == 0 && blocks / s >= 2 && tiles * s <= grid) best = s;
    return best;
}

size_t whole_layer_splitk_bytes(int T, int d) { return static_cast<size_t>(T >> 6) * (d >> 6) * 8 * 4096 * sizeof(float); }

const char* launch_whole_layer(Runtime* rt, WholeLayerArgs a, bool backward, cudaStream_t stream)
{
    const int grid = rt->sm_count;
    const int tiles = (a.T >> 6) * (a.d >> 6);
    a.split_o = pick_slices(tiles, a.d, grid - (a.d >> 6) * (a.d >> 6));
    a.split_fc2 = pick_slices(tiles, a.F, grid);
    a.split_dh2 = pick_slices(tiles, a.F, grid - (a.F >> 6) * (a.d >> 6));
    a.split_dh1 = pick_slices(tiles, 3 * a.d, grid - (3 * a.d >> 6) * (a.d >> 6));
    const cudaError_t e = launch_coop(backward ? whole_layer_bwd_kernel : whole_layer_fwd_kernel, grid, stream, a);
    return e == cudaSuccess ? nullptr : cudaGetErrorString(e);
}

}  // namespace pw
