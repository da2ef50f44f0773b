// Causal attention backward on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// Two kernels so that every output element is owned by exactly one CTA (no atomics; bitwise
// reproducible), after delta = rowsum(dO * O) (attention.cu):
//
//   dkdv : CTA = one 128-key tile j of one (sequence, head); streams 64-query sub-tiles u >= 2j.
//            S^T  = K_j Q_u^T      (128 x 64)   dP^T = V_j dO_u^T   (128 x 64)      -> TMEM, 2 buffers each
//            P^T  = exp2(S^T * scale*log2e - lse*log2e), masked;  dS^T = P^T * (dP^T - delta)
//            dV_j += P^T dO_u      dK_j += dS^T Q_u                                  -> TMEM accumulators
//          P^T / dS^T are written back to TMEM as packed bf16 and fed to the MMA from there; the
//          Q_u / dO_u shared-memory tiles serve both as K-major operands (scores) and as MN-major
//          operands (dV, dK) without any transpose.
//   dq   : CTA = two adjacent 128-query tiles (ping-pong), streams 64-key sub-tiles.
//            S = Q K_v^T (128 x 64), dP = dO V_v^T, dS = P * (dP - delta), dQ += dS K_v.
//
// Warps: 0 = TMA producer, 1 = MMA issuer (+ TMEM allocation), 2..9 = element-wise warps (a warp
// may only touch TMEM lanes 32*(warp%4)..+31; the two warps of a lane quarter split the columns).
// No running maximum is needed: lse from the forward normalises P directly.
// Every mbarrier wait is bounded (see mbar_wait).
#include "pw_kernels.h"

namespace pw {
namespace {

constexpr int kThreads = 320;
constexpr float kLog2e = 1.4426950408889634f;

struct BwdParams {
    int S, H;
    float scale;
    const float* lse;
    const float* delta;
    DeviceStatus* status;
};

// ------------------------------------------------------------------------------------------- dK, dV
template <int DH>
struct KvSmem {
    static constexpr int kBlocks = DH / 64;
    static constexpr int kKV = 128 * DH * 2;                 // K_j or V_j tile
    static constexpr int kSub = 64 * DH * 2;                 // one 64-row sub-tile of Q or dO
    static constexpr int kStages = 4;
    static constexpr int kK = 0, kV = kKV, kQ = 2 * kKV;     // ring: stage s holds Q_u at kQ + s*2*kSub, dO_u right after
    static constexpr int kBars = kQ + kStages * 2 * kSub;
    static constexpr int kBytes = kBars + 256 + 1024;
};

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
attn_bwd_dkdv_tc_kernel(const __grid_constant__ CUtensorMap tmKV,   // qkv, box 64 x 128 rows
                        const __grid_constant__ CUtensorMap tmQ,    // qkv, box 64 x 64 rows
                        const __grid_constant__ CUtensorMap tmDO,   // dout, box 64 x 64 rows
                        const __grid_constant__ CUtensorMap tmOut,  // dqkv, box 64 x 128 rows
                        const BwdParams p)
{
    using L = KvSmem<DH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(sm);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
    // 0 kv_full | 1..4 q_full | 5..8 q_empty | 9,10 st_full | 11,12 p_full | 13 acc_full
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x;                               // key tile; tile 0 has the most query sub-tiles
    const int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
    const int d = p.H * DH;
    const int kv0 = j * 128, row_base = b * p.S;
    const int u0 = 2 * j, n_u = p.S / 64 - u0;              // query sub-tiles u0 .. u0 + n_u - 1

    if (threadIdx.x == 0) {
        for (int i = 0; i < 11; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(11), 256); mbar_init(bar(12), 256);
        mbar_init(bar(13), 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmKV); prefetch_tmap(&tmQ); prefetch_tmap(&tmDO); prefetch_tmap(&tmOut);
    }
    grid_dep_launch();
    grid_dep_wait();                                        // inputs come from the previous kernels
    if (threadIdx.x == 0) {
        // first loads go out before the TMEM allocation and the CTA-wide barrier
        mbar_arrive_expect_tx(bar(0), 2 * L::kKV);
        for (int kb = 0; kb < L::kBlocks; ++kb) {
            tma_load_2d(sbase + L::kK + kb * 16384, &tmKV, d + h * DH + kb * 64, row_base + kv0, bar(0));
            tma_load_2d(sbase + L::kV + kb * 16384, &tmKV, 2 * d + h * DH + kb * 64, row_base + kv0, bar(0));
        }
        for (int i = 0; i < n_u && i < L::kStages; ++i) {
            mbar_arrive_expect_tx(bar(1 + i), 2 * L::kSub);
            const uint32_t qs = sbase + L::kQ + i * 2 * L::kSub, gs = qs + L::kSub;
            for (int kb = 0; kb < L::kBlocks; ++kb) {
                tma_load_2d(qs + kb * 8192, &tmQ, h * DH + kb * 64, row_base + (u0 + i) * 64, bar(1 + i));
                tma_load_2d(gs + kb * 8192, &tmDO, h * DH + kb * 64, row_base + (u0 + i) * 64, bar(1 + i));
            }
        }
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // TMEM columns: S^T buffers at 0 / 64, dP^T buffers at 128 / 192, dV at 256, dK at 384

    if (warp == 0) {
        if (lane == 0) {
            for (int i = L::kStages; i < n_u; ++i) {        // K_j, V_j and the first sub-tiles were requested in the prologue
                const int s = i % L::kStages, ph = (i / L::kStages) & 1;
                if (!mbar_wait(bar(5 + s), ph ^ 1, abort_flag, p.status, 500)) break;
                mbar_arrive_expect_tx(bar(1 + s), 2 * L::kSub);
                const uint32_t qs = sbase + L::kQ + s * 2 * L::kSub, gs = qs + L::kSub;
                const int qrow = row_base + (u0 + i) * 64;
                for (int kb = 0; kb < L::kBlocks; ++kb) {
                    tma_load_2d(qs + kb * 8192, &tmQ, h * DH + kb * 64, qrow, bar(1 + s));
                    tma_load_2d(gs + kb * 8192, &tmDO, h * DH + kb * 64, qrow, bar(1 + s));
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_st = make_idesc_bf16(128, 64, false, false);
            constexpr uint32_t idesc_acc = make_idesc_bf16(128, DH, false, true);
            const uint64_t desc_k = make_smem_desc_sw128(sbase + L::kK, 16, 1024);
            const uint64_t desc_v = make_smem_desc_sw128(sbase + L::kV, 16, 1024);
            auto issue_scores = [&](int i) {                // S^T and dP^T of sub-tile i into buffer i & 1
                const int s = i % L::kStages, hb = i & 1;
                const uint32_t qs = sbase + L::kQ + s * 2 * L::kSub;
                const uint64_t dq = make_smem_desc_sw128(qs, 16, 1024), dg = desc_advance(dq, L::kSub);
                const uint32_t st = tmem_base + hb * 64;
#pragma unroll
                for (int kb = 0; kb < L::kBlocks; ++kb)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_f16(st, desc_advance(desc_k, kb * 16384 + kk * 32), desc_advance(dq, kb * 8192 + kk * 32),
                                 idesc_st, (kb | kk) ? 1u : 0u);
#pragma unroll
                for (int kb = 0; kb < L::kBlocks; ++kb)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_f16(st + 128, desc_advance(desc_v, kb * 16384 + kk * 32), desc_advance(dg, kb * 8192 + kk * 32),
                                 idesc_st, (kb | kk) ? 1u : 0u);
                umma_commit(bar(9 + hb));
            };
            auto issue_acc = [&](int i) {                   // dV += P^T dO_u, dK += dS^T Q_u
                const int s = i % L::kStages, hb = i & 1;
                const uint32_t qs = sbase + L::kQ + s * 2 * L::kSub;
                const uint64_t dq = make_smem_desc_sw128(qs, 8192, 1024), dg = desc_advance(dq, L::kSub);
                const uint32_t pt = tmem_base + hb * 64;
                const uint32_t first = i ? 1u : 0u;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_f16_ta(tmem_base + 256, pt + (ks >> 1) * 32 + (ks & 1) * 8, desc_advance(dg, ks * 2048), idesc_acc,
                                ks ? 1u : first);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_f16_ta(tmem_base + 384, pt + 128 + (ks >> 1) * 32 + (ks & 1) * 8, desc_advance(dq, ks * 2048), idesc_acc,
                                ks ? 1u : first);
                umma_commit(bar(5 + s));                    // Q_u / dO_u stage free
            };
            bool ok = mbar_wait(bar(0), 0, abort_flag, p.status, 510) && mbar_wait(bar(1), 0, abort_flag, p.status, 511);
            if (ok) { tc_fence_after(); issue_scores(0); }
            for (int i = 0; i < n_u && ok; ++i) {
                if (i + 1 < n_u) {
                    const int sn = (i + 1) % L::kStages, phn = ((i + 1) / L::kStages) & 1;
                    if (!mbar_wait(bar(1 + sn), phn, abort_flag, p.status, 512)) { ok = false; break; }
                    tc_fence_after();
                    issue_scores(i + 1);
                }
                if (!mbar_wait(bar(11 + (i & 1)), (i >> 1) & 1, abort_flag, p.status, 513)) { ok = false; break; }
                tc_fence_after();
                issue_acc(i);
            }
            if (ok) umma_commit(bar(13));
        }
    } else {
        const int q = warp & 3, ch = (warp - 2) >> 2;       // lane quarter, column half (32 of the 64 queries)
        const int r = q * 32 + lane;                        // key row inside the tile
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const float sl2 = p.scale * kLog2e;
        const float* lse_row = p.lse + (static_cast<size_t>(b) * p.H + h) * p.S;
        const float* dl_row = p.delta + (static_cast<size_t>(b) * p.H + h) * p.S;
        bool ok = true;
        for (int i = 0; i < n_u; ++i) {
            const int hb = i & 1, qc0 = (u0 + i) * 64 + ch * 32;   // first query column of this thread's slice
            // -lse*log2e and -delta of this slice's 32 queries, as two-wide operands
            uint64_t nl2[16], ndl[16];
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const float4 a = *(reinterpret_cast<const float4*>(lse_row + qc0) + g);
                const float4 c = *(reinterpret_cast<const float4*>(dl_row + qc0) + g);
                nl2[2 * g] = pack_f32x2(-a.x * kLog2e, -a.y * kLog2e); nl2[2 * g + 1] = pack_f32x2(-a.z * kLog2e, -a.w * kLog2e);
                ndl[2 * g] = pack_f32x2(-c.x, -c.y); ndl[2 * g + 1] = pack_f32x2(-c.z, -c.w);
            }
            ok = mbar_wait(bar(9 + hb), (i >> 1) & 1, abort_flag, p.status, 520);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t sv[32], dv[32];
            tmem_ld32(tmem_base + lane_addr + hb * 64 + ch * 32, sv);
            tmem_ld32(tmem_base + lane_addr + 128 + hb * 64 + ch * 32, dv);
            tc_wait_ld();
            const bool diag = qc0 < kv0 + 128;               // some (key, query) pairs of this slice are masked
            uint32_t pp[16], dd[16];
            const uint64_t sl2x2 = pack_f32x2(sl2, sl2);
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
                float a0, a1, d0, d1;
                unpack_f32x2(ffma2(pack_f32x2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1])), sl2x2, nl2[c >> 1]), a0, a1);
                float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                if (diag) {
                    if (qc0 + c < kv0 + r) p0 = 0.f;
                    if (qc0 + c + 1 < kv0 + r) p1 = 0.f;
                }
                const uint64_t pv = pack_f32x2(p0, p1);
                unpack_f32x2(fmul2(pv, fadd2(pack_f32x2(__uint_as_float(dv[c]), __uint_as_float(dv[c + 1])), ndl[c >> 1])), d0, d1);
                pp[c >> 1] = pack_bf16(p0, p1);
                dd[c >> 1] = pack_bf16(d0, d1);
            }
            // packed operands go back into this warp's own columns: P^T over S^T, dS^T over dP^T
            tmem_st16(tmem_base + lane_addr + hb * 64 + ch * 32, pp);
            tmem_st16(tmem_base + lane_addr + 128 + hb * 64 + ch * 32, dd);
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar(11 + hb));
        }
        if (ok) {
            ok = mbar_wait(bar(13), 0, abort_flag, p.status, 521);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            // this warp converts columns [ch*DH/2, +DH/2) of dV and dK and stages them over V_j / K_j
#pragma unroll 1
            for (int which = 0; which < 2; ++which) {
                uint8_t* stage = sm + (which == 0 ? L::kV : L::kK);
                const float mul = which == 0 ? 1.0f : p.scale;
#pragma unroll 1
                for (int c = 0; c < DH / 64; ++c) {
                    const int col0 = ch * (DH / 2) + c * 32;
                    uint32_t v[32];
                    tmem_ld32(tmem_base + lane_addr + 256 + which * 128 + col0, v);
                    tc_wait_ld();
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        float f[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * g + i]) * mul;
                        const int col = col0 + g * 8, blk = col >> 6, chunk = (col & 63) >> 3;
                        *reinterpret_cast<uint4*>(stage + blk * 16384 + r * 128 + ((chunk ^ (r & 7)) << 4)) = pack8(f);
                    }
                }
            }
            fence_proxy_async();
            named_bar_sync(1, 256);
            if (warp == 2 && lane == 0) {
                for (int kb = 0; kb < L::kBlocks; ++kb) {
                    tma_store_2d(&tmOut, sbase + L::kK + kb * 16384, d + h * DH + kb * 64, row_base + kv0);
                    tma_store_2d(&tmOut, sbase + L::kV + kb * 16384, 2 * d + h * DH + kb * 64, row_base + kv0);
                }
                bulk_commit();
                bulk_wait0();
            }
        }
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {}
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------- dQ
template <int DH>
struct DqSmem {
    static constexpr int kBlocks = DH / 64;
    static constexpr int kTile = 128 * DH * 2;               // Q_t or dO_t
    static constexpr int kSub = 64 * DH * 2;                 // 64-key sub-tile of K or V
    static constexpr int kQ = 0;                             // Q_A, Q_B, dO_A, dO_B
    static constexpr int kKV = 4 * kTile;                    // 2 stages x (K_v, V_v)
    static constexpr int kBars = kKV + 4 * kSub;
    static constexpr int kBytes = kBars + 256 + 1024;
};

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
attn_bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tmQ,    // qkv, box 64 x 128 rows
                      const __grid_constant__ CUtensorMap tmDO,   // dout, box 64 x 128 rows
                      const __grid_constant__ CUtensorMap tmKV,   // qkv, box 64 x 64 rows
                      const __grid_constant__ CUtensorMap tmOut,  // dqkv, box 64 x 128 rows
                      const BwdParams p)
{
    using L = DqSmem<DH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(sm);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
    // 0 q_full | 1,2 kv_full | 3,4 kv_empty | 5,6 s_full[t] | 7,8 ds_full[t] | 9,10 acc_full[t]
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pair = gridDim.x - 1 - blockIdx.x;            // heaviest (latest) query tiles first
    const int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
    const int d = p.H * DH;
    const int q0A = pair * 256, q0B = q0A + 128;
    const bool hasB = q0B < p.S;
    const int nA = q0A / 64 + 2, nB = hasB ? nA + 2 : 0;    // 64-key sub-tiles each query tile needs
    const int n_kv = hasB ? nB : nA;
    const int row_base = b * p.S;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 7; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(7), 128); mbar_init(bar(8), 128);
        mbar_init(bar(9), 1); mbar_init(bar(10), 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmQ); prefetch_tmap(&tmDO); prefetch_tmap(&tmKV); prefetch_tmap(&tmOut);
    }
    grid_dep_launch();
    grid_dep_wait();                                        // inputs come from the previous kernels
    if (threadIdx.x == 0) {
        // first loads go out before the TMEM allocation and the CTA-wide barrier
        const int nq = hasB ? 2 : 1;
        mbar_arrive_expect_tx(bar(0), nq * 2 * L::kTile);
        for (int t = 0; t < nq; ++t)
            for (int kb = 0; kb < L::kBlocks; ++kb) {
                tma_load_2d(sbase + L::kQ + t * L::kTile + kb * 16384, &tmQ, h * DH + kb * 64, row_base + q0A + t * 128, bar(0));
                tma_load_2d(sbase + L::kQ + (2 + t) * L::kTile + kb * 16384, &tmDO, h * DH + kb * 64, row_base + q0A + t * 128, bar(0));
            }
        for (int v = 0; v < 2 && v < n_kv; ++v) {
            mbar_arrive_expect_tx(bar(1 + v), 2 * L::kSub);
            const uint32_t ks = sbase + L::kKV + v * 2 * L::kSub, vs = ks + L::kSub;
            for (int kb = 0; kb < L::kBlocks; ++kb) {
                tma_load_2d(ks + kb * 8192, &tmKV, d + h * DH + kb * 64, row_base + v * 64, bar(1 + v));
                tma_load_2d(vs + kb * 8192, &tmKV, 2 * d + h * DH + kb * 64, row_base + v * 64, bar(1 + v));
            }
        }
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // TMEM columns of tile t: S at t*256, dP at t*256 + 64, dQ at t*256 + 128

    if (warp == 0) {
        if (lane == 0) {
            for (int v = 2; v < n_kv; ++v) {                // Q, dO and the first two sub-tiles were requested in the prologue
                const int s = v & 1, ph = (v >> 1) & 1;
                if (!mbar_wait(bar(3 + s), ph ^ 1, abort_flag, p.status, 600)) break;
                mbar_arrive_expect_tx(bar(1 + s), 2 * L::kSub);
                const uint32_t ks = sbase + L::kKV + s * 2 * L::kSub, vs = ks + L::kSub;
                for (int kb = 0; kb < L::kBlocks; ++kb) {
                    tma_load_2d(ks + kb * 8192, &tmKV, d + h * DH + kb * 64, row_base + v * 64, bar(1 + s));
                    tma_load_2d(vs + kb * 8192, &tmKV, 2 * d + h * DH + kb * 64, row_base + v * 64, bar(1 + s));
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_sc = make_idesc_bf16(128, 64, false, false);
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, DH, false, true);
            auto issue_scores = [&](int t, int s) {         // S_t = Q_t K_v^T, dP_t = dO_t V_v^T
                const uint64_t dq = make_smem_desc_sw128(sbase + L::kQ + t * L::kTile, 16, 1024);
                const uint64_t dg = desc_advance(dq, 2 * L::kTile);
                const uint64_t dk = make_smem_desc_sw128(sbase + L::kKV + s * 2 * L::kSub, 16, 1024);
                const uint64_t dv = desc_advance(dk, L::kSub);
                const uint32_t dst = tmem_base + t * 256;
#pragma unroll
                for (int kb = 0; kb < L::kBlocks; ++kb)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_f16(dst, desc_advance(dq, kb * 16384 + kk * 32), desc_advance(dk, kb * 8192 + kk * 32),
                                 idesc_sc, (kb | kk) ? 1u : 0u);
#pragma unroll
                for (int kb = 0; kb < L::kBlocks; ++kb)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_f16(dst + 64, desc_advance(dg, kb * 16384 + kk * 32), desc_advance(dv, kb * 8192 + kk * 32),
                                 idesc_sc, (kb | kk) ? 1u : 0u);
                umma_commit(bar(5 + t));
            };
            auto issue_dq = [&](int t, int s, bool acc) {   // dQ_t += dS_t K_v (dS packed in the S columns)
                const uint64_t dk = make_smem_desc_sw128(sbase + L::kKV + s * 2 * L::kSub, 8192, 1024);
                const uint32_t dst = tmem_base + t * 256 + 128, src = tmem_base + t * 256;
                umma_f16_ta(dst, src, dk, idesc_dq, acc ? 1u : 0u);
#pragma unroll
                for (int kq = 1; kq < 4; ++kq) umma_f16_ta(dst, src + kq * 8, desc_advance(dk, kq * 2048), idesc_dq, 1u);
            };
            bool ok = mbar_wait(bar(0), 0, abort_flag, p.status, 610) && mbar_wait(bar(1), 0, abort_flag, p.status, 611);
            if (ok) {
                tc_fence_after();
                issue_scores(0, 0);
                if (hasB) issue_scores(1, 0);
            }
            for (int v = 0; v < n_kv && ok; ++v) {
                const int s = v & 1, nxt = v + 1, sn = nxt & 1, phn = (nxt >> 1) & 1;
                bool k_waited = false;
                if (v < nA) {
                    if (!mbar_wait(bar(7), v & 1, abort_flag, p.status, 612)) { ok = false; break; }
                    tc_fence_after();
                    issue_dq(0, s, v > 0);
                    if (v == nA - 1) umma_commit(bar(9));
                }
                if (nxt < nA) {
                    if (!mbar_wait(bar(1 + sn), phn, abort_flag, p.status, 613)) { ok = false; break; }
                    k_waited = true;
                    tc_fence_after();
                    issue_scores(0, sn);
                }
                if (v < nB) {
                    if (!mbar_wait(bar(8), v & 1, abort_flag, p.status, 614)) { ok = false; break; }
                    tc_fence_after();
                    issue_dq(1, s, v > 0);
                    if (v == nB - 1) umma_commit(bar(10));
                }
                umma_commit(bar(3 + s));                    // K_v / V_v stage free
                if (nxt < nB) {
                    if (!k_waited && !mbar_wait(bar(1 + sn), phn, abort_flag, p.status, 615)) { ok = false; break; }
                    tc_fence_after();
                    issue_scores(1, sn);
                }
            }
        }
    } else {
        const int t = (warp - 2) >> 2, q = warp & 3;
        const int r = q * 32 + lane;
        const int q0 = t == 0 ? q0A : q0B;
        const int n_t = t == 0 ? nA : nB;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t s_addr = tmem_base + lane_addr + t * 256;
        const float sl2 = p.scale * kLog2e;
        float lse2 = 0.f, dlt = 0.f;
        if (n_t > 0) {
            const size_t idx = (static_cast<size_t>(b) * p.H + h) * p.S + q0 + r;
            lse2 = p.lse[idx] * kLog2e;
            dlt = p.delta[idx];
        }
        bool ok = true;
        for (int v = 0; v < n_t; ++v) {
            ok = mbar_wait(bar(5 + t), v & 1, abort_flag, p.status, 620);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const bool diag = v * 64 + 63 > q0;              // some keys of this sub-tile are masked for some rows
            const uint64_t sl2x2 = pack_f32x2(sl2, sl2), nlse2 = pack_f32x2(-lse2, -lse2), ndlt = pack_f32x2(-dlt, -dlt);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t sv[32], dv[32], ds[16];
                tmem_ld32(s_addr + c * 32, sv);
                tmem_ld32(s_addr + 64 + c * 32, dv);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float a0, a1, d0, d1;
                    unpack_f32x2(ffma2(pack_f32x2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), sl2x2, nlse2), a0, a1);
                    float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                    if (diag) {
                        const int key = v * 64 + c * 32 + i;
                        if (key > q0 + r) p0 = 0.f;
                        if (key + 1 > q0 + r) p1 = 0.f;
                    }
                    unpack_f32x2(fmul2(pack_f32x2(p0, p1), fadd2(pack_f32x2(__uint_as_float(dv[i]), __uint_as_float(dv[i + 1])), ndlt)), d0, d1);
                    ds[i >> 1] = pack_bf16(d0, d1);
                }
                tmem_st16(s_addr + c * 16, ds);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar(7 + t));
        }
        if (ok && n_t > 0) {
            ok = mbar_wait(bar(9 + t), 0, abort_flag, p.status, 621);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok && n_t > 0) {
            tc_fence_after();
            uint8_t* stage = sm + L::kQ + t * L::kTile;     // Q_t is idle now
#pragma unroll 1
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(s_addr + 128 + c * 32, v);
                tc_wait_ld();
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * g + i]) * p.scale;
                    const int col = c * 32 + g * 8, blk = col >> 6, chunk = (col & 63) >> 3;
                    *reinterpret_cast<uint4*>(stage + blk * 16384 + r * 128 + ((chunk ^ (r & 7)) << 4)) = pack8(f);
                }
            }
            fence_proxy_async();
            named_bar_sync(1 + t, 128);
            if ((warp & 3) == 2 && lane == 0) {
                for (int kb = 0; kb < L::kBlocks; ++kb)
                    tma_store_2d(&tmOut, sbase + L::kQ + t * L::kTile + kb * 16384, h * DH + kb * 64, row_base + q0);
                bulk_commit();
                bulk_wait0();
            }
        }
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {}
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 [rows, cols] row-major, box 64 columns x box_rows rows, 128-byte swizzle.
const char* encode_rows(Runtime* rt, CUtensorMap* map, const void* ptr, uint64_t cols, uint64_t rows, uint32_t box_rows)
{
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(rt->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? nullptr : "cuTensorMapEncodeTiled failed";
}

}  // namespace

const char* configure_attention_bwd_tc()
{
    if (cudaFuncSetAttribute(attn_bwd_dkdv_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, KvSmem<64>::kBytes) != cudaSuccess ||
        cudaFuncSetAttribute(attn_bwd_dkdv_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, KvSmem<128>::kBytes) != cudaSuccess)
        return "cudaFuncSetAttribute(attention bwd) failed";
    if (cudaFuncSetAttribute(attn_bwd_dq_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<64>::kBytes) != cudaSuccess ||
        cudaFuncSetAttribute(attn_bwd_dq_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<128>::kBytes) != cudaSuccess)
        return "cudaFuncSetAttribute(attention bwd dq) failed";
    return nullptr;
}

// dQ part of dqkv.
const char* launch_attention_bwd_dq(Runtime* rt, const void* qkv, const void* dout, const void* lse, const void* delta,
                                    int B, int S, int H, int dh, void* dqkv, DeviceStatus* status, cudaStream_t stream)
{
    const int d = H * dh;
    const uint64_t T = static_cast<uint64_t>(B) * S;
    CUtensorMap tmQ, tmDO, tmKV, tmOut;
    const char* e;
    if ((e = encode_rows(rt, &tmQ, qkv, 3ull * d, T, 128))) return e;
    if ((e = encode_rows(rt, &tmDO, dout, d, T, 128))) return e;
    if ((e = encode_rows(rt, &tmKV, qkv, 3ull * d, T, 64))) return e;
    if ((e = encode_rows(rt, &tmOut, dqkv, 3ull * d, T, 128))) return e;
    BwdParams p;
    p.S = S; p.H = H; p.scale = 1.0f / sqrtf(static_cast<float>(dh));
    p.lse = static_cast<const float*>(lse); p.delta = static_cast<const float*>(delta);
    p.status = status;
    dim3 grid((S + 255) / 256, B * H);
    const cudaError_t e2 = dh == 64
        ? launch_k(attn_bwd_dq_tc_kernel<64>, grid, dim3(kThreads), DqSmem<64>::kBytes, stream, tmQ, tmDO, tmKV, tmOut, p)
        : launch_k(attn_bwd_dq_tc_kernel<128>, grid, dim3(kThreads), DqSmem<128>::kBytes, stream, tmQ, tmDO, tmKV, tmOut, p);
    return e2 == cudaSuccess ? nullptr : "attention bwd (dq) launch failed";
}

// dK and dV parts of dqkv.  lse, delta: fp32 [B,H,S].
const char* launch_attention_bwd_dkdv(Runtime* rt, const void* qkv, const void* dout, const void* lse, const void* delta,
                                      int B, int S, int H, int dh, void* dqkv, DeviceStatus* status, cudaStream_t stream)
{
    const int d = H * dh;
    const uint64_t T = static_cast<uint64_t>(B) * S;
    CUtensorMap tmKV, tmQ, tmDO, tmOut;
    const char* e;
    if ((e = encode_rows(rt, &tmKV, qkv, 3ull * d, T, 128))) return e;
    if ((e = encode_rows(rt, &tmQ, qkv, 3ull * d, T, 64))) return e;
    if ((e = encode_rows(rt, &tmDO, dout, d, T, 64))) return e;
    if ((e = encode_rows(rt, &tmOut, dqkv, 3ull * d, T, 128))) return e;
    BwdParams p;
    p.S = S; p.H = H; p.scale = 1.0f / sqrtf(static_cast<float>(dh));
    p.lse = static_cast<const float*>(lse); p.delta = static_cast<const float*>(delta);
    p.status = status;
    dim3 grid(S / 128, B * H);
    const cudaError_t e2 = dh == 64
        ? launch_k(attn_bwd_dkdv_tc_kernel<64>, grid, dim3(kThreads), KvSmem<64>::kBytes, stream, tmKV, tmQ, tmDO, tmOut, p)
        : launch_k(attn_bwd_dkdv_tc_kernel<128>, grid, dim3(kThreads), KvSmem<128>::kBytes, stream, tmKV, tmQ, tmDO, tmOut, p);
    return e2 == cudaSuccess ? nullptr : "attention bwd (dk, dv) launch failed";
}

}  // namespace pw
