// bf16 GEMM for sm_100a: TMA -> 4-stage shared-memory ring -> tcgen05.mma (fp32 accumulators in
// TMEM, double buffered) -> epilogue warps (tcgen05.ld -> bias / GeLU / residual -> global).
//
// One persistent CTA per SM, 6 warps: warp 0 = TMA producer (one lane), warp 1 = MMA issuer (one
// lane; the warp also owns the TMEM allocation), warps 2..5 = epilogue (warp w reads TMEM lanes
// 32*(w%4) .. +31, i.e. 32 rows of the 128-row tile each).  Output tile 128 x 256, K step 64.
//
// Operand layouts are handled without physical transposes: an operand whose contraction index
// is contiguous in memory ("K-major") is loaded as [rows][64 k] boxes, one whose row index is
// contiguous ("MN-major": the weight in dgrad, both operands in wgrad) as [64 k][64 rows] boxes;
// both use the 128-byte swizzle and the matching shared-memory descriptors.
//
// Every wait on an mbarrier is bounded (see mbar_wait); on expiry the CTA raises an abort flag,
// all roles leave their loops, the TMEM allocation is released and the kernel returns.
#include <cstdlib>

#include "pw_kernels.h"

namespace pw {
namespace {

constexpr int BM = 128, BN_MAX = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_TILE_BYTES = BM * BK * 2;       // 16 KB
constexpr int B_TILE_BYTES = BN_MAX * BK * 2;   // 32 KB (a narrower tile uses the front of it)
constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES;
constexpr int EPI_WARPS = 8;
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;   // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int TMEM_COLS = 2 * BN_MAX;           // two accumulators: the whole 512-column TMEM
constexpr int SLAB_BYTES = 4096;                // per epilogue warp: 32 rows x 128 bytes, swizzled
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * SLAB_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct GemmParams {
    int M, N, K;
    int bn;                      // tile width actually used: 128, 192 or 256
    const __nv_bfloat16* bias;
    const __nv_bfloat16* aux_in; int ld_aux;
    int accumulate, act;
    int m_tiles, n_tiles;
    int n_fastest;               // tile numbering: 1 = consecutive tiles share the A row panel, 0 = the B panel
    int split_begin;             // tiles >= split_begin are issued as two units (tail balancing): half-width
                                 // tiles in the one-CTA kernel, halves of the K range in the CTA-pair kernel
    int total_virtual;           // split_begin + 2 * (m_tiles*n_tiles - split_begin)
    float* split_ws;             // CTA-pair kernel: where the K halves leave their partial sums
    float* row_dot; int head_dim, seq_len;   // kEpiRowDot: per (row, head) dot products with aux_in, [B, H, S]
    DeviceStatus* status;
};

// Virtual tile v -> (m0, n0, width).  Tiles that run at the same time should touch as few distinct
// operand panels as possible (they have to sit in L2 together), so the numbering runs fastest along
// the dimension with fewer tiles.  The tiles of the last,
// partly filled round are cut in two half-width tiles so that every SM gets one.
__device__ __forceinline__ void tile_info(const GemmParams& p, int v, int& m0, int& n0, int& bn)
{
    int t = v, half = 0;
    bn = p.bn;
    if (v >= p.split_begin) {
        const int hv = v - p.split_begin;
        t = p.split_begin + (hv >> 1);
        half = hv & 1;
        bn = p.bn >> 1;
    }
    const int mi = p.n_fastest ? t / p.n_tiles : t % p.m_tiles;
    const int ni = p.n_fastest ? t % p.n_tiles : t / p.m_tiles;
    m0 = mi * BM;
    n0 = ni * p.bn + half * (p.bn >> 1);
}

// One 8-column group of the bf16 epilogues: f = acc (+bias) (+residual | x GeLU'(u)).  `aux` holds the
// group's 8 residual / pre-activation values, fetched by the caller ahead of the TMEM load.
template <int EPI>
__device__ __forceinline__ void epilogue_group(const uint32_t* v, int row, int c, const GemmParams& p, const uint4& aux, float* f)
{
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[j]);
    if (c < p.N) {
        if constexpr (EPI == kEpiBias || EPI == kEpiBiasResid || EPI == kEpiBiasGelu) {
            float b[8];
            unpack8(*(reinterpret_cast<const uint4*>(p.bias + c)), b);
#pragma unroll
            for (int j = 0; j < 8; ++j) f[j] += b[j];
        }
        if constexpr (EPI == kEpiBiasResid) {
            if (row < p.M) {
                float r[8];
                unpack8(aux, r);
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] += r[j];
            }
        }
        if constexpr (EPI == kEpiDGelu) {
            if (row < p.M) {
                float u[8];
                unpack8(aux, u);
                if (p.act == 0) {                           // one uniform branch per group, not per pair
#pragma unroll
                    for (int j = 0; j < 8; j += 2) gelu_grad_mul2_erf(f[j], f[j + 1], u[j], u[j + 1]);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; j += 2) gelu_grad_mul2(f[j], f[j + 1], u[j], u[j + 1], p.act);
                }
            }
        }
    }
}

// Epilogue of one accumulator tile for one warp: TMEM -> registers -> swizzled shared slab -> TMA
// store (rows >= M and columns >= N are clipped by the tensor map).  `taddr` addresses this warp's
// lane quarter of the accumulator, row0 is the first of its 32 rows, pi selects which of the two
// warps of the quarter it is (they take alternate column chunks).
// Partial sums of one 32 x 32 accumulator chunk as the K halves of a cut tile exchange them: eight
// 512-byte rows of [lane][4 floats], so that every access of a warp is one contiguous 512 bytes.
__device__ __forceinline__ void add_partner_chunk(uint32_t (&v)[32], const float* partner_chunk, int lane)
{
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 t = __ldcg(reinterpret_cast<const float4*>(partner_chunk + i * 128 + lane * 4));
        v[4 * i] = __float_as_uint(__uint_as_float(v[4 * i]) + t.x);
        v[4 * i + 1] = __float_as_uint(__uint_as_float(v[4 * i + 1]) + t.y);
        v[4 * i + 2] = __float_as_uint(__uint_as_float(v[4 * i + 2]) + t.z);
        v[4 * i + 3] = __float_as_uint(__uint_as_float(v[4 * i + 3]) + t.w);
    }
}

template <int EPI, bool SINGLE_SLAB = false, bool SPLIT = false>
__device__ __forceinline__ void epilogue_tile(uint32_t taddr, int row0, int n0, int bn, int pi, int pstride, int lane,
                                              uint8_t* slab, uint32_t slab_u32, uint32_t& nout, const CUtensorMap* tmC,
                                              const CUtensorMap* tmAux, const GemmParams& p,
                                              const float* partner = nullptr /* SPLIT: the other K half's partial sums, [chunk][1024] */)
{
    const int row = row0 + lane;
    uint8_t* my_row = slab + lane * 128;
    if constexpr (EPI == kEpiF32) {
        const int nsteps = bn / 32;
#pragma unroll 1
        for (int s = pi; s < nsteps; s += pstride) {
            const int col0 = n0 + s * 32;
            if (col0 >= p.N) break;
            uint32_t v[32];
            tmem_ld32(taddr + s * 32, v);
            tc_wait_ld();
            if constexpr (SPLIT) add_partner_chunk(v, partner + s * 1024, lane);
            if (lane == 0) bulk_wait_read0();
            __syncwarp();
#pragma unroll
            for (int g = 0; g < 8; ++g)
                *reinterpret_cast<uint4*>(my_row + ((g ^ (lane & 7)) << 4)) =
                    make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                if (p.accumulate) tma_reduce_add_2d(tmC, slab_u32, col0, row0);
                else tma_store_2d(tmC, slab_u32, col0, row0);
                bulk_commit();
            }
        }
    } else {
        // 32 columns per chunk; the slab is two 2 KB halves (32 rows x 64 bytes, 64-byte
        // swizzle) used alternately, so one store is always in flight behind the math.
        const int nchunks = bn / 32;
        const uint32_t sw = (lane >> 1) & 3;
        // The warps of a lane quarter take alternate chunks - except with the row-dot epilogue, where each
        // takes a run of neighbouring chunks, so that all columns of a head meet in one thread.
        const int ch_first = EPI == kEpiRowDot ? pi * (nchunks / pstride) : pi;
        const int ch_step = EPI == kEpiRowDot ? 1 : pstride;
        const int ch_end = EPI == kEpiRowDot ? ch_first + nchunks / pstride : nchunks;
        float dot = 0.f;
#pragma unroll 1
        for (int ch = ch_first; ch < ch_end; ch += ch_step) {
            const int col0 = n0 + ch * 32;
            if (col0 >= p.N) break;
            // residual / saved pre-activation of this chunk: requested before the TMEM load so that the
            // (row-strided, L2-latency) reads overlap it
            uint4 aux[4] = {};
            if constexpr (EPI == kEpiBiasResid || EPI == kEpiDGelu || EPI == kEpiRowDot) {
                if (row < p.M) {
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        if (col0 + g * 8 < p.N)
                            aux[g] = *reinterpret_cast<const uint4*>(p.aux_in + static_cast<size_t>(row) * p.ld_aux + col0 + g * 8);
                }
            }
            uint32_t v[32];
            tmem_ld32(taddr + ch * 32, v);
            tc_wait_ld();
            if constexpr (SPLIT) add_partner_chunk(v, partner + ch * 1024, lane);
            uint4 o[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                float f[8];
                epilogue_group<EPI>(v + 8 * g, row, col0 + g * 8, p, aux[g], f);
                o[g] = pack8(f);
                if constexpr (EPI == kEpiRowDot) {
                    float r[8];
                    unpack8(aux[g], r);                      // zeros beyond M and N
#pragma unroll
                    for (int j = 0; j < 8; ++j) dot = fmaf(f[j], r[j], dot);
                }
                if constexpr (EPI == kEpiBiasGelu) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[8 * g + j] = __float_as_uint(f[j]);   // fp32 pre-activation, kept for GeLU
                }
            }
            auto store_chunk = [&](const uint4* src, const CUtensorMap* map) {
                const uint32_t half = SINGLE_SLAB ? 0u : (nout++ & 1u) * 2048u;
                if (lane == 0) { if (SINGLE_SLAB) bulk_wait_read0(); else bulk_wait_read1(); }
                __syncwarp();
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    *reinterpret_cast<uint4*>(slab + half + lane * 64 + ((g ^ sw) << 4)) = src[g];
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(map, slab_u32 + half, col0, row0);
                    bulk_commit();
                }
            };
            store_chunk(o, tmC);
            if constexpr (EPI == kEpiRowDot) {
                if ((col0 + 32) % p.head_dim == 0) {         // last chunk of a head: its row sums are complete
                    if (row < p.M) {
                        const int b = row / p.seq_len, sq = row - b * p.seq_len, h = col0 / p.head_dim;
                        p.row_dot[(static_cast<size_t>(b) * (p.N / p.head_dim) + h) * p.seq_len + sq] = dot;
                    }
                    dot = 0.f;
                }
            }
            if constexpr (EPI == kEpiBiasGelu) {
                // GeLU of the fp32 pre-activation, evaluated while the store above drains the slab
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float f[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[8 * g + j]);
                    if (p.act == 0) {                       // one uniform branch per group, not per pair
#pragma unroll
                        for (int j = 0; j < 8; j += 2) gelu2_erf(f[j], f[j + 1]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; j += 2) gelu2(f[j], f[j + 1], p.act);
                    }
                    o[g] = pack8(f);
                }
                store_chunk(o, tmAux);
            }
        }
    }
}

template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmBh /* B with a half-width box */,
            const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmAux, const GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* slabs = tiles + STAGES * STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(slabs + EPI_WARPS * SLAB_BYTES);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STAGES);
    const uint32_t accf0 = smem_u32(bars + 2 * STAGES), acce0 = smem_u32(bars + 2 * STAGES + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_k = (p.K + BK - 1) / BK;
    const int total_tiles = p.total_virtual;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 32 * EPI_WARPS); }
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        prefetch_tmap(&tmC);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    grid_dep_launch();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_wait();                                    // inputs of this GEMM come from the previous kernel

    if (warp == 0) {
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int m0, n0, bn;
                tile_info(p, tile, m0, n0, bn);
                const uint32_t stage_tx = A_TILE_BYTES + bn * BK * 2;
                const CUtensorMap* mapB = bn == p.bn ? &tmB : &tmBh;
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 100)) { ok = false; break; }
                    const uint32_t fb = full0 + 8 * stage;
                    mbar_arrive_expect_tx(fb, stage_tx);
                    const uint32_t a_dst = smem_u32(tiles + stage * STAGE_BYTES), b_dst = a_dst + A_TILE_BYTES;
                    if constexpr (!A_MN) {
                        tma_load_2d(a_dst, &tmA, kb * BK, m0, fb);
                    } else {
#pragma unroll
                        for (int j = 0; j < BM / 64; ++j) tma_load_2d(a_dst + j * 8192, &tmA, m0 + 64 * j, kb * BK, fb);
                    }
                    if constexpr (!B_MN) {
                        tma_load_2d(b_dst, mapB, kb * BK, n0, fb);
                    } else {
                        for (int j = 0; j < bn / 64; ++j) tma_load_2d(b_dst + j * 8192, &tmB, n0 + 64 * j, kb * BK, fb);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc_full = make_idesc_bf16(BM, p.bn, A_MN, B_MN);
            const uint32_t idesc_half = make_idesc_bf16(BM, p.bn >> 1, A_MN, B_MN);
            uint32_t stage = 0, phase = 0, it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
                const uint32_t idesc = tile >= p.split_begin ? idesc_half : idesc_full;
                const uint32_t buf = it & 1, acc_phase = (it >> 1) & 1;
                if (!mbar_wait(acce0 + 8 * buf, acc_phase ^ 1, abort_flag, p.status, 200)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN_MAX;
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 201)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_base = smem_u32(tiles + stage * STAGE_BYTES), b_base = a_base + A_TILE_BYTES;
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                        // K-major: 16 k = 32 bytes along the swizzled 128-byte row; 8-row groups 1024 B apart.
                        // MN-major: 16 k = two 8-k groups of 1024 B; 64-row groups 8192 B apart.
                        const uint64_t adesc = A_MN ? make_smem_desc_sw128(a_base + kk * 2048, 8192, 1024)
                                                    : make_smem_desc_sw128(a_base + kk * 32, 16, 1024);
                        const uint64_t bdesc = B_MN ? make_smem_desc_sw128(b_base + kk * 2048, 8192, 1024)
                                                    : make_smem_desc_sw128(b_base + kk * 32, 16, 1024);
                        umma_f16(d_tmem, adesc, bdesc, idesc, (kb | kk) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty0 + 8 * stage);   // frees the stage once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit(accf0 + 8 * buf);  // accumulator complete
            }
        }
    } else {
        // Epilogue: warp w may read TMEM lanes 32*(w%4)..+31; the two warps of a lane quarter take
        // alternate column steps.  Each step goes TMEM -> registers -> swizzled shared slab -> one
        // TMA store (rows >= M and columns >= N are clipped by the tensor map).
        const int q = warp & 3, pi = (warp - 2) >> 2;
        uint8_t* slab = slabs + (warp - 2) * SLAB_BYTES;
        const uint32_t slab_u32 = smem_u32(slab);
        uint32_t it = 0, nout = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
            int m0, n0, bn;
            tile_info(p, tile, m0, n0, bn);
            const uint32_t buf = it & 1, acc_phase = (it >> 1) & 1;
            bool ok = mbar_wait(accf0 + 8 * buf, acc_phase, abort_flag, p.status, 300);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * BN_MAX;
            epilogue_tile<EPI>(taddr, m0 + q * 32, n0, bn, pi, 2, lane, slab, slab_u32, nout, &tmC, &tmAux, p);
            tc_fence_before();
            mbar_arrive(acce0 + 8 * buf);
        }
        if (lane == 0) bulk_wait0();
    }

    __syncwarp();
    if (*abort_flag) {   // give copies and MMAs still in flight time to land before releasing anything
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {}
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2): a cluster of two CTAs computes one 256 x bn tile.  CTA r of the
// pair loads its own 128 rows of A and its own half (bn/2 rows) of B - with plain per-CTA TMA loads
// whose bytes are credited to the leader's "full" barrier - and the leader CTA issues one M = 256
// MMA that reads both CTAs' shared memory and writes each CTA's 128 x bn accumulator into that
// CTA's own TMEM.  Per FLOP this moves a third less data into shared memory than the one-CTA tile
// and makes 128-wide tiles affordable, which removes most of the wave-quantisation loss on the
// N = d_model GEMMs.  Barriers: full[s] (leader, 1 arrival + both CTAs' bytes), empty[s] and
// acc_full[b] (one in each CTA, signalled by the leader's tcgen05.commit to both), acc_empty[b]
// (leader, one arrival per epilogue warp of both CTAs).
// The epilogues that evaluate GeLU / GeLU' are instruction-bound with 8 warps (two per scheduler),
// so those instantiations run 16 epilogue warps and use one 2 KB output slab per warp instead of two.
constexpr int P_STAGE_BYTES = 32768;            // A: 128 x 64 (16 KB) + B half: up to 128 x 64 (16 KB)
template <int EPI> struct PairCfg {
    static constexpr int kEpiWarps = (EPI == kEpiBiasGelu || EPI == kEpiDGelu) ? 16 : 8;
    static constexpr int kStages = 6;
    static constexpr int kSlab = kEpiWarps == 16 ? 2048 : SLAB_BYTES;   // 16 warps: one 2 KB slab each, no ping-pong
    static constexpr int kThreads = 64 + 32 * kEpiWarps;
    static constexpr int kSmem = kStages * P_STAGE_BYTES + kEpiWarps * kSlab + 1024 + 256;
};

// Work unit v of the CTA-pair kernel: a whole tile, or - for the tiles of a thin last round - one
// half of a tile's K range (slot = which cut tile, half = which half).
struct PairUnit { int tile, kb0, kb1, slot, half; };
__device__ __forceinline__ PairUnit pair_unit(const GemmParams& p, int v, int num_k)
{
    PairUnit u;
    if (v < p.split_begin) { u.tile = v; u.kb0 = 0; u.kb1 = num_k; u.slot = -1; u.half = 0; return u; }
    const int hv = v - p.split_begin;
    u.slot = hv >> 1; u.half = hv & 1; u.tile = p.split_begin + u.slot;
    u.kb0 = u.half ? num_k / 2 : 0;
    u.kb1 = u.half ? num_k : num_k / 2;
    return u;
}

template <bool A_MN, bool B_MN, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PairCfg<EPI>::kThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmAux, const GemmParams p)
{
    constexpr int P_STAGES = PairCfg<EPI>::kStages, NEPI = PairCfg<EPI>::kEpiWarps;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* slabs = tiles + P_STAGES * P_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(slabs + NEPI * PairCfg<EPI>::kSlab);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + P_STAGES);
    const uint32_t accf0 = smem_u32(bars + 2 * P_STAGES), acce0 = smem_u32(bars + 2 * P_STAGES + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * P_STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = leader
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int num_k = (p.K + BK - 1) / BK;
    const int total_tiles = p.total_virtual;            // work units: whole pair tiles (m_tiles counts 256-row blocks) + K halves
    const int bn = p.bn, half_n = bn >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 2 * NEPI); }
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        prefetch_tmap(&tmC);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    grid_dep_launch();
    cluster_sync_all();                                 // both CTAs' barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_wait();                                    // inputs of this GEMM come from the previous kernel

    if (warp == 0) {
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            const uint32_t pair_tx = 2u * (A_TILE_BYTES + half_n * BK * 2);
            for (int unit = pair_id; unit < total_tiles && ok; unit += n_pairs) {
                const PairUnit un = pair_unit(p, unit, num_k);
                const int tile = un.tile;
                const int mi = p.n_fastest ? tile / p.n_tiles : tile % p.m_tiles;
                const int ni = p.n_fastest ? tile % p.n_tiles : tile / p.m_tiles;
                const int m0 = mi * 256 + rank * 128;
                const int n0 = ni * bn + rank * half_n;
                for (int kb = un.kb0; kb < un.kb1; ++kb) {
                    if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 700)) { ok = false; break; }
                    const uint32_t fb = mapa_shared(full0 + 8 * stage, 0);     // the leader's barrier
                    if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * stage, pair_tx);
                    const uint32_t a_dst = smem_u32(tiles + stage * P_STAGE_BYTES), b_dst = a_dst + A_TILE_BYTES;
                    if constexpr (!A_MN) {
                        tma_load_2d_pair(a_dst, &tmA, kb * BK, m0, fb);
                    } else {
#pragma unroll
                        for (int j = 0; j < 2; ++j) tma_load_2d_pair(a_dst + j * 8192, &tmA, m0 + 64 * j, kb * BK, fb);
                    }
                    if constexpr (!B_MN) {
                        tma_load_2d_pair(b_dst, &tmB, kb * BK, n0, fb);
                    } else {
                        for (int j = 0; j < half_n / 64; ++j) tma_load_2d_pair(b_dst + j * 8192, &tmB, n0 + 64 * j, kb * BK, fb);
                    }
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = make_idesc_bf16(256, bn, A_MN, B_MN);
            uint32_t stage = 0, phase = 0, it = 0;
            bool ok = true;
            for (int unit = pair_id; unit < total_tiles && ok; unit += n_pairs, ++it) {
                const PairUnit un = pair_unit(p, unit, num_k);
                const uint32_t buf = it & 1, acc_phase = (it >> 1) & 1;
                if (!mbar_wait(acce0 + 8 * buf, acc_phase ^ 1, abort_flag, p.status, 710)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN_MAX;
                for (int kb = un.kb0; kb < un.kb1; ++kb) {
                    if (!mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 711)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_base = smem_u32(tiles + stage * P_STAGE_BYTES), b_base = a_base + A_TILE_BYTES;
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                        const uint64_t adesc = A_MN ? make_smem_desc_sw128(a_base + kk * 2048, 8192, 1024)
                                                    : make_smem_desc_sw128(a_base + kk * 32, 16, 1024);
                        const uint64_t bdesc = B_MN ? make_smem_desc_sw128(b_base + kk * 2048, 8192, 1024)
                                                    : make_smem_desc_sw128(b_base + kk * 32, 16, 1024);
                        umma_f16_pair(d_tmem, adesc, bdesc, idesc, (kb != un.kb0 || kk != 0) ? 1u : 0u);
                    }
                    umma_commit_pair(empty0 + 8 * stage, 3);     // frees the stage in both CTAs
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit_pair(accf0 + 8 * buf, 3);     // both CTAs' accumulators complete
            }
        }
    } else {
        const int q = warp & 3, pi = (warp - 2) >> 2;
        uint8_t* slab = slabs + (warp - 2) * PairCfg<EPI>::kSlab;
        const uint32_t slab_u32 = smem_u32(slab);
        uint32_t it = 0, nout = 0;
        for (int unit = pair_id; unit < total_tiles; unit += n_pairs, ++it) {
            const PairUnit un = pair_unit(p, unit, num_k);
            const int tile = un.tile;
            const int mi = p.n_fastest ? tile / p.n_tiles : tile % p.m_tiles;
            const int ni = p.n_fastest ? tile % p.n_tiles : tile / p.m_tiles;
            const int m0 = mi * 256 + rank * 128, n0 = ni * bn;
            const uint32_t buf = it & 1, acc_phase = (it >> 1) & 1;
            bool ok = mbar_wait(accf0 + 8 * buf, acc_phase, abort_flag, p.status, 720);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * BN_MAX;
            if (EPI == kEpiF32 || un.slot < 0) {                 // (the fp32-output GEMMs are never cut)
                epilogue_tile<EPI, NEPI == 16>(taddr, m0 + q * 32, n0, bn, pi, NEPI / 4, lane, slab, slab_u32, nout, &tmC, &tmAux, p);
            } else {
                // Half of a cut tile's K range.  Every epilogue warp leaves its part of the partial sums in
                // the scratch, then draws a ticket shared with the same warp of the CTA that has the
                // other half: the first of the two is finished, the second adds the first one's sums
                // to its own (fp32, two addends: the result does not depend on who came first) and
                // runs the epilogue.  Nobody waits for anybody.
                const int nchunks = bn / 32;
                const size_t region = static_cast<size_t>(nchunks) * 1024;       // floats per (slot, half, rank, quarter)
                float* mine = p.split_ws + ((((static_cast<size_t>(un.slot) * 2 + un.half) * 2 + rank) * 4) + q) * region;
                const float* other = p.split_ws + ((((static_cast<size_t>(un.slot) * 2 + (un.half ^ 1)) * 2 + rank) * 4) + q) * region;
#pragma unroll 1
                for (int ch = pi; ch < nchunks; ch += NEPI / 4) {
                    if (n0 + ch * 32 >= p.N) break;
                    uint32_t v[32];
                    tmem_ld32(taddr + ch * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        __stcg(reinterpret_cast<float4*>(mine + ch * 1024 + i * 128 + lane * 4),
                               make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]), __uint_as_float(v[4 * i + 2]),
                                           __uint_as_float(v[4 * i + 3])));
                }
                __threadfence();
                __syncwarp();
                int* ticket = &p.status->tickets[(un.slot * 2 + static_cast<int>(rank)) * 16 + (warp - 2)];
                int before = 0;
                if (lane == 0) before = atomicAdd(ticket, 1);
                before = __shfl_sync(0xffffffffu, before, 0);
                if (before != 0) {
                    if (lane == 0) *ticket = 0;                                  // both halves have drawn: ready for the next launch
                    __threadfence();
                    epilogue_tile<EPI, NEPI == 16, true>(taddr, m0 + q * 32, n0, bn, pi, NEPI / 4, lane, slab, slab_u32, nout, &tmC, &tmAux, p, other);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(acce0 + 8 * buf, 0));
        }
        if (lane == 0) bulk_wait0();
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {}
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                 // neither CTA releases TMEM or exits while its peer may still touch it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D tensor map (bf16, or fp32 when f32 is set): `inner` contiguous elements per row, `outer`
// rows, row pitch ld elements; 128-byte swizzle, so box_inner * element size must be 128 bytes.
const char* encode_2d(Runtime* rt, CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t outer, uint64_t ld,
                      uint32_t box_inner, uint32_t box_outer, bool f32 = false, bool swizzle64 = false)
{
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {ld * (f32 ? 4 : 2)};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(rt->encode_tiled)(
        map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? nullptr : "cuTensorMapEncodeTiled failed";
}

template <bool A_MN, bool B_MN, int EPI>
const char* launch_inst(Runtime* rt, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmBh,
                        const CUtensorMap& tmC, const CUtensorMap& tmAux, const GemmParams& p, cudaStream_t stream)
{
    auto kern = gemm_kernel<A_MN, B_MN, EPI>;
    const int total = p.m_tiles * p.n_tiles;
    const int grid = total < rt->sm_count ? total : rt->sm_count;
    return launch_k(kern, dim3(grid), dim3(GEMM_THREADS), SMEM_BYTES, stream, tmA, tmB, tmBh, tmC, tmAux, p) == cudaSuccess
               ? nullptr : "gemm launch failed";
}

template <bool A_MN, bool B_MN, int EPI>
const char* launch_pair(Runtime* rt, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                        const CUtensorMap& tmAux, const GemmParams& p, cudaStream_t stream)
{
    auto kern = gemm_pair_kernel<A_MN, B_MN, EPI>;
    const int total = p.total_virtual;
    const int max_pairs = rt->sm_count / 2;
    const int pairs = total < max_pairs ? total : max_pairs;
    return launch_k(kern, dim3(2 * pairs), dim3(PairCfg<EPI>::kThreads), PairCfg<EPI>::kSmem, stream, tmA, tmB, tmC, tmAux, p) == cudaSuccess
               ? nullptr : "gemm (CTA pair) launch failed";
}

template <bool A_MN, bool B_MN, int EPI>
bool set_attr()
{
    return cudaFuncSetAttribute(gemm_kernel<A_MN, B_MN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                SMEM_BYTES) == cudaSuccess &&
           cudaFuncSetAttribute(gemm_pair_kernel<A_MN, B_MN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                PairCfg<EPI>::kSmem) == cudaSuccess;
}

}  // namespace

// Opt every instantiation into its dynamic shared-memory size, once per process (never on the
// enqueue path, so a stream capture sees launches only).
const char* configure_gemm()
{
    const bool ok = set_attr<false, false, kEpiNone>() && set_attr<false, false, kEpiBias>() &&
                    set_attr<false, false, kEpiBiasResid>() && set_attr<false, false, kEpiBiasGelu>() &&
                    set_attr<false, true, kEpiNone>() && set_attr<false, true, kEpiDGelu>() && set_attr<false, true, kEpiRowDot>() &&
                    set_attr<true, true, kEpiF32>();
    return ok ? nullptr : "cudaFuncSetAttribute(gemm) failed";
}

static const char* launch_gemm_pair(Runtime* rt, const GemmArgs& a, DeviceStatus* status, cudaStream_t stream)
{
    const bool a_mn = a.layout == kNT, b_mn = a.layout == kNN || a.layout == kNT;
    const bool f32_out = a.epilogue == kEpiF32;
    const int m_tiles = (a.M + 255) / 256, pairs = rt->sm_count / 2;
    // Tile width: 256 unless the rounds it needs waste more than a 128-wide tiling does (a
    // 128-wide pair tile moves as many operand bytes per FLOP as the one-CTA 256-wide tile).
    int bn = 256;
    {
        const int forced = tuning().gemm_bn;
        auto cost = [&](int w) {
            const long long tiles = static_cast<long long>(m_tiles) * ((a.N + w - 1) / w);
            const long long rounds = (tiles + pairs - 1) / pairs;
            return static_cast<double>(rounds) * w * (w == 128 ? 1.6 : 1.0);   // 128-wide pair tiles measured ~1.6x slower per FLOP
        };
        if (cost(128) < cost(256)) bn = 128;
        if (forced == 128 || forced == 256) bn = forced;
        if (a.epilogue == kEpiRowDot) bn = 256;              // an epilogue warp must own whole heads (128 columns)
    }
    CUtensorMap tmA, tmB, tmC, tmAux;
    const char* e;
    e = a_mn ? encode_2d(rt, &tmA, a.A, a.M, a.K, a.lda, 64, BK) : encode_2d(rt, &tmA, a.A, a.K, a.M, a.lda, BK, BM);
    if (e) return e;
    e = b_mn ? encode_2d(rt, &tmB, a.B, a.N, a.K, a.ldb, 64, BK) : encode_2d(rt, &tmB, a.B, a.K, a.N, a.ldb, BK, bn / 2);
    if (e) return e;
    e = encode_2d(rt, &tmC, a.C, a.N, a.M, a.ldc, 32, 32, f32_out, !f32_out);
    if (e) return e;
    e = encode_2d(rt, &tmAux, a.epilogue == kEpiBiasGelu ? a.aux_out : a.C, a.N, a.M, a.ldc, 32, 32, f32_out, !f32_out);
    if (e) return e;
    GemmParams p;
    p.M = a.M; p.N = a.N; p.K = a.K; p.bn = bn;
    p.bias = static_cast<const __nv_bfloat16*>(a.bias);
    p.aux_in = static_cast<const __nv_bfloat16*>(a.aux_in); p.ld_aux = a.ld_aux;
    p.accumulate = a.accumulate; p.act = a.act;
    p.m_tiles = m_tiles; p.n_tiles = (a.N + bn - 1) / bn;
    p.split_begin = p.m_tiles * p.n_tiles; p.total_virtual = p.split_begin;
    p.split_ws = nullptr;
    p.row_dot = static_cast<float*>(a.row_dot); p.head_dim = a.head_dim; p.seq_len = a.seq_len;
    {
        // Tail balancing: when the last round of tiles would keep at most half of the CTA pairs busy,
        // each of its tiles becomes two units of half the K range (needs the caller's scratch).
        const bool no_split = tuning().gemm_split == 0;
        const int total = p.m_tiles * p.n_tiles, num_k = (a.K + BK - 1) / BK;
        const int rem = total % pairs;
        const int min_k = tuning().gemm_split_min_k;
        // (short K ranges lose more to the second prologue and epilogue than the idle half round costs)
        if (a.split_ws && !no_split && !f32_out && a.epilogue != kEpiRowDot && total > pairs && rem > 0 && 2 * rem <= pairs && rem <= kSplitMaxTiles &&
            num_k >= min_k) {
            p.split_begin = total - rem;
            p.total_virtual = p.split_begin + 2 * rem;
            p.split_ws = static_cast<float*>(a.split_ws);
        }
    }
    p.n_fastest = p.n_tiles < p.m_tiles ? 1 : 0;
    p.status = status;
    const int key = a.layout * 16 + a.epilogue;
    switch (key) {
        case kTN * 16 + kEpiNone: return launch_pair<false, false, kEpiNone>(rt, tmA, tmB, tmC, tmAux, p, stream);
        case kTN * 16 + kEpiBias: return launch_pair<false, false, kEpiBias>(rt, tmA, tmB, tmC, tmAux, p, stream);
        case kTN * 16 + kEpiBiasResid: return launch_pair<false, false, kEpiBiasResid>(rt, tmA, tmB, tmC, tmAux, p, stream);
        case kTN * 16 + kEpiBiasGelu: return launch_pair<false, false, kEpiBiasGelu>(rt, tmA, tmB, tmC, tmAux, p, stream);
        case kNN * 16 + kEpiNone: return launch_pair<false, true, kEpiNone>(rt, tmA, tmB, tmC, tmAux, p, stream);
        case kNN * 16 + kEpiDGelu: return launch_pair<false, true, kEpiDGelu>(rt, tmA, tmB, tmC, tmAux, p, stream);
        case kNN * 16 + kEpiRowDot: return launch_pair<false, true, kEpiRowDot>(rt, tmA, tmB, tmC, tmAux, p, stream);
        case kNT * 16 + kEpiF32: return launch_pair<true, true, kEpiF32>(rt, tmA, tmB, tmC, tmAux, p, stream);
        default: return "gemm: unsupported layout/epilogue combination";
    }
}

// Scratch for the K halves of cut tiles: (cut tile, half, CTA of the pair) x 128 rows x 256 columns, fp32.
size_t gemm_split_ws_bytes() { return static_cast<size_t>(kSplitMaxTiles) * 2 * 2 * 128 * BN_MAX * sizeof(float); }

const char* launch_gemm(Runtime* rt, const GemmArgs& a, DeviceStatus* status, cudaStream_t stream)
{
    if (a.M <= 0 || a.N <= 0 || a.K <= 0) return "gemm: non-positive dimension";
    if ((a.M % 8) || (a.N % 8) || (a.K % 8)) return "gemm: M, N, K must be multiples of 8";
    if ((a.lda % 8) || (a.ldb % 8) || (a.ldc % 8)) return "gemm: leading dimensions must be multiples of 8";
    auto misaligned = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) != 0; };
    if (!a.A || !a.B || !a.C || misaligned(a.A) || misaligned(a.B) || misaligned(a.C)) return "gemm: null or misaligned operand";
    const bool need_bias = a.epilogue == kEpiBias || a.epilogue == kEpiBiasResid || a.epilogue == kEpiBiasGelu;
    const bool need_aux_in = a.epilogue == kEpiBiasResid || a.epilogue == kEpiDGelu || a.epilogue == kEpiRowDot;
    if (a.epilogue == kEpiRowDot &&
        (!a.row_dot || (a.head_dim != 64 && a.head_dim != 128) || (a.N % a.head_dim) || a.seq_len <= 0 || (a.M % a.seq_len)))
        return "gemm: the row-dot epilogue needs an output, head_dim 64 or 128 dividing N, and seq_len dividing M";
    if (need_bias && (!a.bias || misaligned(a.bias))) return "gemm: epilogue needs a 16-byte aligned bias";
    if (need_aux_in && (!a.aux_in || misaligned(a.aux_in) || (a.ld_aux % 8))) return "gemm: epilogue needs aux_in";
    if (a.epilogue == kEpiBiasGelu && (!a.aux_out || misaligned(a.aux_out))) return "gemm: epilogue needs aux_out";

    const bool a_mn = a.layout == kNT, b_mn = a.layout == kNN || a.layout == kNT;
    const bool f32_out = a.epilogue == kEpiF32;
    const int pair_mode = tuning().gemm_pair;
    if (pair_mode && a.M >= 256) return launch_gemm_pair(rt, a, status, stream);
    if (f32_out && (a.ldc % 4)) return "gemm: fp32 ldc must be a multiple of 4";
    // Tile width: the one that needs the least (rounds x width) on this many SMs; ties go to the
    // wider tile (less operand traffic per FLOP).
    const int m_tiles = (a.M + BM - 1) / BM;
    // Tile width 256 unless that leaves most SMs without a tile (small problems are latency-bound;
    // a narrower tile spreads them over more SMs).  Narrower tiles cost more operand traffic per
    // FLOP and were measured slower whenever every SM already has work.
    int bn = BN_MAX;
    while (bn > 128 && static_cast<long long>(m_tiles) * ((a.N + bn - 1) / bn) * 2 <= rt->sm_count) bn -= 64;
    {
        const int forced = tuning().gemm_bn;
        if (forced == 128 || forced == 192 || forced == 256) bn = forced;
        if (a.epilogue == kEpiRowDot) bn = BN_MAX;           // an epilogue warp must own whole heads (128 columns)
    }
    CUtensorMap tmA, tmB, tmBh, tmC, tmAux;
    const char* e;
    // K-major operand [rows, K]: box 64 k x rows.  MN-major operand stored [K, rows]: box 64 rows x 64 k.
    e = a_mn ? encode_2d(rt, &tmA, a.A, a.M, a.K, a.lda, 64, BK) : encode_2d(rt, &tmA, a.A, a.K, a.M, a.lda, BK, BM);
    if (e) return e;
    e = b_mn ? encode_2d(rt, &tmB, a.B, a.N, a.K, a.ldb, 64, BK) : encode_2d(rt, &tmB, a.B, a.K, a.N, a.ldb, BK, bn);
    if (e) return e;
    e = b_mn ? encode_2d(rt, &tmBh, a.B, a.N, a.K, a.ldb, 64, BK) : encode_2d(rt, &tmBh, a.B, a.K, a.N, a.ldb, BK, bn / 2);
    if (e) return e;

    // Output maps: a store box is 32 rows x 32 columns (fp32: 128-byte rows, 128-byte swizzle;
    // bf16: 64-byte rows, 64-byte swizzle).
    e = encode_2d(rt, &tmC, a.C, a.N, a.M, a.ldc, 32, 32, f32_out, !f32_out);
    if (e) return e;
    e = encode_2d(rt, &tmAux, a.epilogue == kEpiBiasGelu ? a.aux_out : a.C, a.N, a.M, a.ldc, 32, 32, f32_out, !f32_out);
    if (e) return e;

    GemmParams p;
    p.M = a.M; p.N = a.N; p.K = a.K; p.bn = bn;
    p.bias = static_cast<const __nv_bfloat16*>(a.bias);
    p.aux_in = static_cast<const __nv_bfloat16*>(a.aux_in); p.ld_aux = a.ld_aux;
    p.accumulate = a.accumulate; p.act = a.act;
    p.m_tiles = m_tiles; p.n_tiles = (a.N + bn - 1) / bn;
    p.n_fastest = p.n_tiles < p.m_tiles ? 1 : 0;
    p.status = status;
    p.split_ws = nullptr;
    p.row_dot = static_cast<float*>(a.row_dot); p.head_dim = a.head_dim; p.seq_len = a.seq_len;
    {
        // Tail balancing: when the last round would leave at least half of the SMs idle, its
        // tiles are issued as two half-width tiles each.
        const int total = p.m_tiles * p.n_tiles;
        const int grid = total < rt->sm_count ? total : rt->sm_count;
        const int rem = total % grid;
        const bool no_split = tuning().gemm_split == 0;
        p.split_begin = total;
        if (bn == BN_MAX && rem > 0 && 2 * rem <= grid && !no_split && a.epilogue != kEpiRowDot) p.split_begin = total - rem;
        p.total_virtual = p.split_begin + 2 * (total - p.split_begin);
    }

    const int key = a.layout * 16 + a.epilogue;
    switch (key) {
        case kTN * 16 + kEpiNone: return launch_inst<false, false, kEpiNone>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        case kTN * 16 + kEpiBias: return launch_inst<false, false, kEpiBias>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        case kTN * 16 + kEpiBiasResid: return launch_inst<false, false, kEpiBiasResid>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        case kTN * 16 + kEpiBiasGelu: return launch_inst<false, false, kEpiBiasGelu>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        case kNN * 16 + kEpiNone: return launch_inst<false, true, kEpiNone>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        case kNN * 16 + kEpiDGelu: return launch_inst<false, true, kEpiDGelu>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        case kNN * 16 + kEpiRowDot: return launch_inst<false, true, kEpiRowDot>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        case kNT * 16 + kEpiF32: return launch_inst<true, true, kEpiF32>(rt, tmA, tmB, tmBh, tmC, tmAux, p, stream);
        default: return "gemm: unsupported layout/epilogue combination";
    }
}

}  // namespace pw
