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
constexpr int kDqThreads = 576;                            // producer warp, MMA warp, 2 x 8 element-wise warps
constexpr float kLog2e = 1.4426950408889634f;


struct BwdParams {
    int S, H, B;
    int tiles_per_seq;          // dQ: pairs of query tiles; dK/dV: key tiles
    int n_items;                // B * H * tiles_per_seq
    float scale;
    const float* lse;
    const float* delta;
    DeviceStatus* status;
    int* sched;                 // {next ticket, CTAs done} of this kernel
};

// ------------------------------------------------------------------------------------------- dK, dV
template <int DH>
struct KvSmem {
    static constexpr int kBlocks = DH / 64;
    static constexpr int kKV = 128 * DH * 2;                 // K_j or V_j tile
    static constexpr int kSub = 64 * DH * 2;                 // one 64-row sub-tile of Q or dO
    static constexpr int kStages = DH == 64 ? 5 : 3;         // Q_u / dO_u ring (the scores run kBufs - 1 sub-tiles ahead of the accumulation)
    static constexpr int kBufs = DH == 64 ? 3 : 2;           // S^T / dP^T buffers in TMEM: with 64-wide heads dV and dK leave room for a third pair
    // TMEM columns: S^T buffer b at 64 b, dP^T buffer b at kDP + 64 b, then dV and dK (DH columns each)
    static constexpr int kDP = 64 * kBufs, kDV = 128 * kBufs, kDK = kDV + (DH == 64 ? 64 : 128);
    // barriers: 0,1 kv_full[buffer] | 2,3 kv_empty[buffer] | kQF+s q_full[stage] | kQE+s q_empty[stage] | kSF+b st_full[b]
    //   kPF+b p_full[b] (256 arrivals) | kAF acc_full | kAE acc_empty (256 arrivals) | kIF+i item_full | kIE+i item_empty (9 arrivals)
    static constexpr int kQF = 4, kQE = kQF + kStages, kSF = kQE + kStages, kPF = kSF + kBufs, kAF = kPF + kBufs, kAE = kAF + 1,
                         kIF = kAE + 1, kIE = kIF + 2, kNumBars = kIE + 2;
    static constexpr int kK = 0;                             // item buffer i: K_j at i*2*kKV, V_j right after (two buffers)
    static constexpr int kQ = 4 * kKV;                       // ring: stage s holds Q_u at kQ + s*2*kSub, dO_u right after
    static constexpr int kBars = kQ + kStages * 2 * kSub;
    static constexpr int kBytes = kBars + 256 + 1024;
};

// Work items of the dK/dV kernel: one per (sequence, head, 128-key tile), heaviest first (key tile
// 0 sees every query), drawn from a global counter by the producer thread.
struct KvItem { int b, h, j, n_u; };
__device__ __forceinline__ bool kv_item(const BwdParams& p, int idx, KvItem& it)
{
    if (idx >= p.n_items) return false;
    const int BH = p.B * p.H;
    const int bh = idx % BH;
    it.j = idx / BH;
    it.b = bh / p.H; it.h = bh % p.H;
    it.n_u = p.S / 64 - 2 * it.j;                           // query sub-tiles 2j .. S/64 - 1
    return true;
}

// Persistent: K_j / V_j are double-buffered across items (the finished item's buffer doubles as the
// staging area of its dK / dV store while the next item's tiles are already in the other one); the
// Q_u / dO_u ring, the S^T / dP^T buffers and every barrier phase run on across item boundaries.
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
    // (barrier map: see KvSmem)
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * i; };
    static_assert(L::kNumBars <= 28, "barriers and the words behind them share 256 bytes");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 28);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* item_slot = reinterpret_cast<volatile int*>(tmem_slot + 2);   // two entries
    auto draw = [&]() {
        const int idx = atomicAdd(p.sched, 1);
        if (idx >= p.n_items && atomicAdd(p.sched + 1, 1) == static_cast<int>(gridDim.x) - 1) {
            p.sched[0] = 0; p.sched[1] = 0;
            __threadfence();
        }
        return idx;
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d = p.H * DH;

    auto load_kv = [&](const KvItem& it, int buf) {
        mbar_arrive_expect_tx(bar(0 + buf), 2 * L::kKV);
        const uint32_t ks = sbase + L::kK + buf * 2 * L::kKV, vs = ks + L::kKV;
        for (int kb = 0; kb < L::kBlocks; ++kb) {
            tma_load_2d(ks + kb * 16384, &tmKV, d + it.h * DH + kb * 64, it.b * p.S + it.j * 128, bar(0 + buf));
            tma_load_2d(vs + kb * 16384, &tmKV, 2 * d + it.h * DH + kb * 64, it.b * p.S + it.j * 128, bar(0 + buf));
        }
    };
    auto load_q = [&](const KvItem& it, int i, int s) {     // Q_u and dO_u, u = 2j + i
        mbar_arrive_expect_tx(bar(L::kQF + s), 2 * L::kSub);
        const uint32_t qs = sbase + L::kQ + s * 2 * L::kSub, gs = qs + L::kSub;
        const int qrow = it.b * p.S + (2 * it.j + i) * 64;
        for (int kb = 0; kb < L::kBlocks; ++kb) {
            tma_load_2d(qs + kb * 8192, &tmQ, it.h * DH + kb * 64, qrow, bar(L::kQF + s));
            tma_load_2d(gs + kb * 8192, &tmDO, it.h * DH + kb * 64, qrow, bar(L::kQF + s));
        }
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kPF; ++i) mbar_init(bar(i), 1);
        for (int i = 0; i < L::kBufs; ++i) mbar_init(bar(L::kPF + i), 256);
        mbar_init(bar(L::kAF), 1);
        mbar_init(bar(L::kAE), 256);
        mbar_init(bar(L::kIF), 1); mbar_init(bar(L::kIF + 1), 1);
        mbar_init(bar(L::kIE), 9); mbar_init(bar(L::kIE + 1), 9);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmKV); prefetch_tmap(&tmQ); prefetch_tmap(&tmDO); prefetch_tmap(&tmOut);
    }
    grid_dep_launch();
    grid_dep_wait();                                        // inputs come from the previous kernels
    int early = 0;                                          // sub-tiles of the first item requested in the prologue
    if (threadIdx.x == 0) {
        KvItem it;
        const int idx0 = draw();
        item_slot[0] = idx0;
        mbar_arrive(bar(L::kIF));
        if (kv_item(p, idx0, it)) {
            load_kv(it, 0);
            for (; early < it.n_u && early < L::kStages; ++early) load_q(it, early, early);
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

    if (warp == 0) {
        if (lane == 0) {
            uint32_t m = 0;                                 // sub-tiles requested so far
            bool ok = true;
            KvItem it;
            int idx = item_slot[0];
            for (int k = 0; ok && kv_item(p, idx, it); ++k) {
                if (k > 0) {
                    if (!mbar_wait(bar(2 + (k & 1)), ((k >> 1) & 1) ^ 1, abort_flag, p.status, 501)) break;
                    load_kv(it, k & 1);
                }
                for (int i = 0; i < it.n_u && ok; ++i, ++m) {
                    if (k == 0 && i < early) continue;
                    const int s = m % L::kStages;
                    if (!mbar_wait(bar(L::kQE + s), ((m / L::kStages) & 1) ^ 1, abort_flag, p.status, 500)) { ok = false; break; }
                    load_q(it, i, s);
                }
                if (!ok) break;
                const int kn = k + 1;
                if (!mbar_wait(bar(L::kIE + (kn & 1)), ((kn >> 1) & 1) ^ 1, abort_flag, p.status, 502)) break;
                idx = draw();
                item_slot[kn & 1] = idx;
                mbar_arrive(bar(L::kIF + (kn & 1)));
            }
        }
    } else if (warp == 1) {
        // converged warp, one elected lane issues (see the forward kernel)
        constexpr uint32_t idesc_st = make_idesc_bf16(128, 64, false, false);
        constexpr uint32_t idesc_acc = make_idesc_bf16(128, DH, false, true);
        const uint32_t tb = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t sb = __shfl_sync(0xffffffffu, sbase, 0);
        auto issue_scores = [&](uint32_t g, int buf) {      // S^T and dP^T of stream position g into buffer g % kBufs
            const int s = g % L::kStages, hb = g % L::kBufs;
            const uint64_t desc_k = make_smem_desc_sw128(sb + L::kK + buf * 2 * L::kKV, 16, 1024);
            const uint64_t desc_v = desc_advance(desc_k, L::kKV);
            const uint64_t dq = make_smem_desc_sw128(sb + L::kQ + s * 2 * L::kSub, 16, 1024), dg = desc_advance(dq, L::kSub);
            const uint32_t st = tb + hb * 64;
            if (elect_one()) {
                // the two products are independent accumulation chains: their steps alternate, so that a step
                // never has to wait for the one before it to leave the pipe
#pragma unroll
                for (int kb = 0; kb < L::kBlocks; ++kb)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        umma_f16(st, desc_advance(desc_k, kb * 16384 + kk * 32), desc_advance(dq, kb * 8192 + kk * 32),
                                 idesc_st, (kb | kk) ? 1u : 0u);
                        umma_f16(st + L::kDP, desc_advance(desc_v, kb * 16384 + kk * 32), desc_advance(dg, kb * 8192 + kk * 32),
                                 idesc_st, (kb | kk) ? 1u : 0u);
                    }
                umma_commit(bar(L::kSF + hb));
            }
            __syncwarp();
        };
        auto issue_acc = [&](uint32_t g, bool first) {      // dV += P^T dO_u, dK += dS^T Q_u
            const int s = g % L::kStages, hb = g % L::kBufs;
            const uint64_t dq = make_smem_desc_sw128(sb + L::kQ + s * 2 * L::kSub, 8192, 1024), dg = desc_advance(dq, L::kSub);
            const uint32_t pt = tb + hb * 64;
            const uint32_t acc0 = first ? 0u : 1u;
            if (elect_one()) {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {             // dV and dK alternate (independent accumulators)
                    umma_f16_ta(tb + L::kDV, pt + (ks >> 1) * 32 + (ks & 1) * 8, desc_advance(dg, ks * 2048), idesc_acc,
                                ks ? 1u : acc0);
                    umma_f16_ta(tb + L::kDK, pt + L::kDP + (ks >> 1) * 32 + (ks & 1) * 8, desc_advance(dq, ks * 2048), idesc_acc,
                                ks ? 1u : acc0);
                }
                umma_commit(bar(L::kQE + s));               // Q_u / dO_u stage free
            }
            __syncwarp();
        };
        auto wait = [&](int b, uint32_t parity, int site) {
            const bool w = mbar_wait(bar(b), parity, abort_flag, p.status, site);
            return __all_sync(0xffffffffu, w);
        };
        uint32_t g0 = 0;                                    // stream position of this item's first sub-tile
        bool ok = true;
        KvItem it;
        for (int k = 0; ok; ++k) {
            if (!wait(L::kIF + (k & 1), (k >> 1) & 1, 514)) break;
            const int idx = __shfl_sync(0xffffffffu, item_slot[k & 1], 0);   // broadcast: everything derived from it is warp-uniform
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(L::kIE + (k & 1)));
            if (!kv_item(p, idx, it)) break;
            const int buf = k & 1, n_u = it.n_u;
            // the scores run kBufs - 1 sub-tiles ahead of the accumulation products
            constexpr int kAhead = L::kBufs - 1;
            ok = wait(0 + buf, (k >> 1) & 1, 510);
            for (int a = 0; a < kAhead && a < n_u && ok; ++a) {
                const uint32_t ga = g0 + a;
                ok = wait(L::kQF + ga % L::kStages, (ga / L::kStages) & 1, 511);
                if (!ok) break;
                tc_fence_after();
                issue_scores(ga, buf);
            }
            if (!ok) break;
            for (int i = 0; i < n_u && ok; ++i) {
                const uint32_t g = g0 + i;
                if (i + kAhead < n_u) {
                    const uint32_t gn = g + kAhead;
                    if (!wait(L::kQF + gn % L::kStages, (gn / L::kStages) & 1, 512)) { ok = false; break; }
                    tc_fence_after();
                    issue_scores(gn, buf);
                }
                if (!wait(L::kPF + g % L::kBufs, (g / L::kBufs) & 1, 513)) { ok = false; break; }
                // the previous item's dV / dK must have been read out before they are overwritten
                if (i == 0 && !wait(L::kAE, (k & 1) ^ 1, 515)) { ok = false; break; }
                tc_fence_after();
                issue_acc(g, i == 0);
            }
            if (!ok) break;
            if (elect_one()) umma_commit(bar(L::kAF));
            __syncwarp();
            g0 += n_u;
        }
    } else {
        const int q = warp & 3, ch = (warp - 2) >> 2;       // lane quarter, column half (32 of the 64 queries)
        const int r = q * 32 + lane;                        // key row inside the tile
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const float sl2 = p.scale * kLog2e;
        uint32_t g = 0;                                     // stream position
        bool ok = true;
        KvItem it;
        for (int k = 0; ok; ++k) {
            ok = mbar_wait(bar(L::kIF + (k & 1)), (k >> 1) & 1, abort_flag, p.status, 522);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int idx = item_slot[k & 1];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(L::kIE + (k & 1)));
            if (!kv_item(p, idx, it)) break;
            const int kv0 = it.j * 128, u0 = 2 * it.j;
            const float* lse_row = p.lse + (static_cast<size_t>(it.b) * p.H + it.h) * p.S;
            const float* dl_row = p.delta + (static_cast<size_t>(it.b) * p.H + it.h) * p.S;
            for (int i = 0; i < it.n_u; ++i, ++g) {
                const int hb = g % L::kBufs, qc0 = (u0 + i) * 64 + ch * 32;   // first query column of this thread's slice
                // -lse*log2e and -delta of this slice's 32 queries, as two-wide operands
                uint64_t nl2[16], ndl[16];
#pragma unroll
                for (int gg = 0; gg < 8; ++gg) {
                    const float4 a = *(reinterpret_cast<const float4*>(lse_row + qc0) + gg);
                    const float4 c = *(reinterpret_cast<const float4*>(dl_row + qc0) + gg);
                    nl2[2 * gg] = pack_f32x2(-a.x * kLog2e, -a.y * kLog2e); nl2[2 * gg + 1] = pack_f32x2(-a.z * kLog2e, -a.w * kLog2e);
                    ndl[2 * gg] = pack_f32x2(-c.x, -c.y); ndl[2 * gg + 1] = pack_f32x2(-c.z, -c.w);
                }
                ok = mbar_wait(bar(L::kSF + hb), (g / L::kBufs) & 1, abort_flag, p.status, 520);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t sv[32], dv[32];
                tmem_ld32(tmem_base + lane_addr + hb * 64 + ch * 32, sv);
                tmem_ld32(tmem_base + lane_addr + L::kDP + hb * 64 + ch * 32, dv);
                tc_wait_ld();
                const bool diag = qc0 < kv0 + 128;           // some (key, query) pairs of this slice are masked
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
                tmem_st16(tmem_base + lane_addr + L::kDP + hb * 64 + ch * 32, dd);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(L::kPF + hb));
            }
            if (ok) {
                ok = mbar_wait(bar(L::kAF), k & 1, abort_flag, p.status, 521);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (!ok) break;
            tc_fence_after();
            // this warp converts columns [ch*DH/2, +DH/2) of dV and dK and stages them over V_j / K_j
            const int buf = k & 1;
#pragma unroll 1
            for (int which = 0; which < 2; ++which) {
                uint8_t* stage = sm + L::kK + buf * 2 * L::kKV + (which == 0 ? L::kKV : 0);
                const float mul = which == 0 ? 1.0f : p.scale;
#pragma unroll 1
                for (int c = 0; c < DH / 64; ++c) {
                    const int col0 = ch * (DH / 2) + c * 32;
                    uint32_t v[32];
                    tmem_ld32(tmem_base + lane_addr + (which == 0 ? L::kDV : L::kDK) + col0, v);
                    tc_wait_ld();
                    if (which == 1 && c == DH / 64 - 1) {    // dV and dK have left TMEM: the next item may overwrite them
                        tc_fence_before();
                        mbar_arrive(bar(L::kAE));
                    }
#pragma unroll
                    for (int gq = 0; gq < 4; ++gq) {
                        float f[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[8 * gq + e]) * mul;
                        const int col = col0 + gq * 8, blk = col >> 6, chunk = (col & 63) >> 3;
                        *reinterpret_cast<uint4*>(stage + blk * 16384 + r * 128 + ((chunk ^ (r & 7)) << 4)) = pack8(f);
                    }
                }
            }
            fence_proxy_async();
            named_bar_sync(1, 256);
            if (warp == 2 && lane == 0) {
                const uint32_t ks = sbase + L::kK + buf * 2 * L::kKV, vs = ks + L::kKV;
                for (int kb = 0; kb < L::kBlocks; ++kb) {
                    tma_store_2d(&tmOut, ks + kb * 16384, d + it.h * DH + kb * 64, it.b * p.S + kv0);
                    tma_store_2d(&tmOut, vs + kb * 16384, 2 * d + it.h * DH + kb * 64, it.b * p.S + kv0);
                }
                bulk_commit();
                bulk_wait_read0();                          // the buffer may take another item's K / V
                mbar_arrive(bar(2 + buf));
            }
        }
        if (warp == 2 && lane == 0) bulk_wait0();
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
    static constexpr int kOut = kKV + 4 * kSub;              // dQ staging tile (shared by both query tiles)
    static constexpr int kBars = kOut + kTile;
    static constexpr int kBytes = kBars + 256 + 1024;
};

// Work items of the dQ kernel: one per (sequence, head, pair of query tiles), heaviest first, drawn
// from a global counter by the producer thread (same scheme as the forward kernel).
struct DqItem { int b, h, q0A, nA, nB; };
__device__ __forceinline__ bool dq_item(const BwdParams& p, int idx, DqItem& it)
{
    if (idx >= p.n_items) return false;
    const int BH = p.B * p.H;
    const int pair = p.tiles_per_seq - 1 - idx / BH, bh = idx % BH;
    it.b = bh / p.H; it.h = bh % p.H;
    it.q0A = pair * 256;
    it.nA = it.q0A / 64 + 2;                                // 64-key sub-tiles each query tile needs
    it.nB = it.q0A + 128 < p.S ? it.nA + 2 : 0;
    return true;
}

template <int DH>
__global__ void __launch_bounds__(kDqThreads, 1)
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
    // barrier map (t = query tile, s = ring stage):
    //   0+t q_full | 2+t q_empty | 4+s kv_full | 6+s kv_empty | 8+t s_full | 10+t ds_full (256 arrivals)
    //   12+t acc_full | 14+t acc_empty (256 arrivals) | 16 staging free | 17+i item_full | 19+i item_empty (17 arrivals)
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 22);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* item_slot = reinterpret_cast<volatile int*>(tmem_slot + 2);   // two entries
    // draws the next item number; past the end, counts this CTA as done and lets the last one clear the counters
    auto draw = [&]() {
        const int idx = atomicAdd(p.sched, 1);
        if (idx >= p.n_items && atomicAdd(p.sched + 1, 1) == static_cast<int>(gridDim.x) - 1) {
            p.sched[0] = 0; p.sched[1] = 0;
            __threadfence();
        }
        return idx;
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d = p.H * DH;

    auto load_q = [&](const DqItem& it, int t) {            // Q_t and dO_t
        mbar_arrive_expect_tx(bar(0 + t), 2 * L::kTile);
        for (int kb = 0; kb < L::kBlocks; ++kb) {
            tma_load_2d(sbase + L::kQ + t * L::kTile + kb * 16384, &tmQ, it.h * DH + kb * 64, it.b * p.S + it.q0A + t * 128, bar(0 + t));
            tma_load_2d(sbase + L::kQ + (2 + t) * L::kTile + kb * 16384, &tmDO, it.h * DH + kb * 64, it.b * p.S + it.q0A + t * 128, bar(0 + t));
        }
    };
    auto load_kv = [&](const DqItem& it, int v, int s) {    // K_v and V_v (64 keys)
        mbar_arrive_expect_tx(bar(4 + s), 2 * L::kSub);
        const uint32_t ks = sbase + L::kKV + s * 2 * L::kSub, vs = ks + L::kSub;
        for (int kb = 0; kb < L::kBlocks; ++kb) {
            tma_load_2d(ks + kb * 8192, &tmKV, d + it.h * DH + kb * 64, it.b * p.S + v * 64, bar(4 + s));
            tma_load_2d(vs + kb * 8192, &tmKV, 2 * d + it.h * DH + kb * 64, it.b * p.S + v * 64, bar(4 + s));
        }
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < 10; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(10), 256); mbar_init(bar(11), 256);
        mbar_init(bar(12), 1); mbar_init(bar(13), 1);
        mbar_init(bar(14), 256); mbar_init(bar(15), 256);
        mbar_init(bar(16), 1);
        mbar_init(bar(17), 1); mbar_init(bar(18), 1);
        mbar_init(bar(19), 17); mbar_init(bar(20), 17);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmQ); prefetch_tmap(&tmDO); prefetch_tmap(&tmKV); prefetch_tmap(&tmOut);
    }
    grid_dep_launch();
    grid_dep_wait();                                        // inputs come from the previous kernels
    if (threadIdx.x == 0) {
        // the first item's first loads go out before the TMEM allocation and the CTA-wide barrier
        DqItem it;
        const int idx0 = draw();
        item_slot[0] = idx0;
        mbar_arrive(bar(17));
        if (dq_item(p, idx0, it)) {
            load_kv(it, 0, 0);
            load_q(it, 0);
            if (it.nB) load_q(it, 1);
            load_kv(it, 1, 1);
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
            uint32_t n = 0;                                 // key sub-tiles requested so far
            uint32_t qn[2] = {0, 0};                        // items each query tile took part in
            bool ok = true;
            DqItem it;
            int idx = item_slot[0];
            for (int k = 0; ok && dq_item(p, idx, it); ++k) {
                const int n_kv = it.nB ? it.nB : it.nA;
                for (int v = 0; v < n_kv && ok; ++v, ++n) {
                    const int s = n & 1;
                    const uint32_t ph = (n >> 1) & 1;
                    const bool early = k == 0 && v < 2;     // requested in the prologue
                    if (!early) {
                        if (!mbar_wait(bar(6 + s), ph ^ 1, abort_flag, p.status, 600)) { ok = false; break; }
                        load_kv(it, v, s);
                    }
                    if (v == 0) {
                        // Q_t / dO_t follow the first key sub-tile; their buffers are free once the
                        // previous item's last scores of tile t have been computed
                        for (int t = 0; t < (it.nB ? 2 : 1) && ok; ++t) {
                            if (k > 0) {
                                if (!mbar_wait(bar(2 + t), (qn[t] & 1) ^ 1, abort_flag, p.status, 601)) { ok = false; break; }
                                load_q(it, t);
                            }
                            ++qn[t];
                        }
                    }
                }
                if (!ok) break;
                const int kn = k + 1;
                if (!mbar_wait(bar(19 + (kn & 1)), ((kn >> 1) & 1) ^ 1, abort_flag, p.status, 602)) break;
                idx = draw();
                item_slot[kn & 1] = idx;
                mbar_arrive(bar(17 + (kn & 1)));
            }
        }
    } else if (warp == 1) {
        // converged warp, one elected lane issues (see the forward kernel)
        constexpr uint32_t idesc_sc = make_idesc_bf16(128, 64, false, false);
        constexpr uint32_t idesc_dq = make_idesc_bf16(128, DH, false, true);
        const uint32_t tb = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t sb = __shfl_sync(0xffffffffu, sbase, 0);
        auto issue_scores = [&](int t, int s) {             // S_t = Q_t K_v^T, dP_t = dO_t V_v^T
            const uint64_t dq = make_smem_desc_sw128(sb + L::kQ + t * L::kTile, 16, 1024);
            const uint64_t dg = desc_advance(dq, 2 * L::kTile);
            const uint64_t dk = make_smem_desc_sw128(sb + L::kKV + s * 2 * L::kSub, 16, 1024);
            const uint64_t dv = desc_advance(dk, L::kSub);
            const uint32_t dst = tb + t * 256;
            if (elect_one()) {
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
                umma_commit(bar(8 + t));
            }
            __syncwarp();
        };
        auto issue_dq = [&](int t, int s, bool acc) {       // dQ_t += dS_t K_v (dS packed in the S columns)
            const uint64_t dk = make_smem_desc_sw128(sb + L::kKV + s * 2 * L::kSub, 8192, 1024);
            const uint32_t dst = tb + t * 256 + 128, src = tb + t * 256;
            if (elect_one()) {
                // dS packed bf16: keys 0..31 in columns 0..15 of S_t, keys 32..63 in columns 32..47
                umma_f16_ta(dst, src, dk, idesc_dq, acc ? 1u : 0u);
#pragma unroll
                for (int kq = 1; kq < 4; ++kq)
                    umma_f16_ta(dst, src + (kq >> 1) * 32 + (kq & 1) * 8, desc_advance(dk, kq * 2048), idesc_dq, 1u);
            }
            __syncwarp();
        };
        auto commit = [&](int b) {
            if (elect_one()) umma_commit(bar(b));
            __syncwarp();
        };
        auto wait = [&](int b, uint32_t parity, int site) {
            const bool w = mbar_wait(bar(b), parity, abort_flag, p.status, site);
            return __all_sync(0xffffffffu, w);
        };
        uint32_t n = 0;                                     // key sub-tiles consumed before this item
        uint32_t nd[2] = {0, 0};                            // dS tiles consumed per query tile
        uint32_t qn[2] = {0, 0};                            // items each query tile took part in
        bool ok = true;
        DqItem it;
        for (int k = 0; ok; ++k) {
            if (!wait(17 + (k & 1), (k >> 1) & 1, 616)) break;
            const int idx = __shfl_sync(0xffffffffu, item_slot[k & 1], 0);   // broadcast: everything derived from it is warp-uniform
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(19 + (k & 1)));
            if (!dq_item(p, idx, it)) break;
            const int nA = it.nA, nB = it.nB, n_kv = nB ? nB : nA;
            {
                const int s = n & 1;
                const uint32_t ph = (n >> 1) & 1;
                ok = wait(4 + s, ph, 611) && wait(0, qn[0] & 1, 610);
                if (!ok) break;
                tc_fence_after();
                issue_scores(0, s);
                if (nB) {
                    if (!wait(1, qn[1] & 1, 617)) { ok = false; break; }
                    tc_fence_after();
                    issue_scores(1, s);
                }
            }
            for (int v = 0; v < n_kv && ok; ++v) {
                const uint32_t nv = n + v, nn = nv + 1;
                const int s = nv & 1, sn = nn & 1;
                const uint32_t phn = (nn >> 1) & 1;
                bool k_waited = false;
                if (v < nA) {
                    if (!wait(10, nd[0] & 1, 612)) { ok = false; break; }
                    ++nd[0];
                    // the previous item's dQ_A must have been read out before it is overwritten
                    if (v == 0 && !wait(14, (qn[0] & 1) ^ 1, 618)) { ok = false; break; }
                    tc_fence_after();
                    issue_dq(0, s, v > 0);
                    if (v == nA - 1) commit(12);
                }
                if (v + 1 < nA) {
                    if (!wait(4 + sn, phn, 613)) { ok = false; break; }
                    k_waited = true;
                    tc_fence_after();
                    issue_scores(0, sn);
                    if (v + 2 == nA) commit(2);             // Q_A / dO_A are not needed again
                }
                if (v < nB) {
                    if (!wait(11, nd[1] & 1, 614)) { ok = false; break; }
                    ++nd[1];
                    if (v == 0 && !wait(15, (qn[1] & 1) ^ 1, 619)) { ok = false; break; }
                    tc_fence_after();
                    issue_dq(1, s, v > 0);
                    if (v == nB - 1) commit(13);
                }
                commit(6 + s);                              // K_v / V_v stage free
                if (v + 1 < nB) {
                    if (!k_waited && !wait(4 + sn, phn, 615)) { ok = false; break; }
                    tc_fence_after();
                    issue_scores(1, sn);
                    if (v + 2 == nB) commit(3);
                }
            }
            n += n_kv;
            ++qn[0];
            if (nB) ++qn[1];
        }
    } else {
        // Element-wise: two threads per query row.  Warps 2..9 serve tile A, 10..17 tile B; the lane
        // quarter is warp % 4, the key half hf = (warp - 2) / 4 % 2: a thread owns 32 of the
        // sub-tile's 64 keys and writes its packed dS over its own S columns.
        const int t = (warp - 2) >> 3, hf = ((warp - 2) >> 2) & 1, q = warp & 3;
        const int r = q * 32 + lane;
        const bool leader = hf == 0 && q == 2 && lane == 0;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t s_addr = tmem_base + lane_addr + t * 256 + hf * 32;       // my S columns; dP is 64 further
        const uint32_t o_addr = tmem_base + lane_addr + t * 256 + 128 + hf * (DH / 2);
        const float sl2 = p.scale * kLog2e;
        uint32_t ns = 0, qn = 0;                            // score tiles and items this query tile has seen
        uint32_t u_base = 0;                                // uses of the staging tile before this item
        bool ok = true;
        DqItem it;
        for (int k = 0; ok; ++k) {
            ok = mbar_wait(bar(17 + (k & 1)), (k >> 1) & 1, abort_flag, p.status, 622);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int idx = item_slot[k & 1];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(19 + (k & 1)));
            if (!dq_item(p, idx, it)) break;
            const int n_t = t == 0 ? it.nA : it.nB;
            const uint32_t u = u_base + t;                  // staging order: A(k), B(k), A(k+1), ...
            u_base += it.nB ? 2 : 1;
            if (n_t == 0) continue;
            const int q0 = it.q0A + t * 128;
            const size_t row_idx = (static_cast<size_t>(it.b) * p.H + it.h) * p.S + q0 + r;
            const float lse2 = p.lse[row_idx] * kLog2e, dlt = p.delta[row_idx];
            const uint64_t sl2x2 = pack_f32x2(sl2, sl2), nlse2 = pack_f32x2(-lse2, -lse2), ndlt = pack_f32x2(-dlt, -dlt);
            for (int v = 0; v < n_t; ++v, ++ns) {
                ok = mbar_wait(bar(8 + t), ns & 1, abort_flag, p.status, 620);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const int key0 = v * 64 + hf * 32;            // first key of my slice
                const bool diag = key0 + 31 > q0;            // some keys of this slice are masked for some rows
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t sv[16], dv[16], ds[8];
                    tmem_ld16(s_addr + c * 16, sv);
                    tmem_ld16(s_addr + 64 + c * 16, dv);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float a0, a1, d0, d1;
                        unpack_f32x2(ffma2(pack_f32x2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), sl2x2, nlse2), a0, a1);
                        float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                        if (diag) {
                            const int key = key0 + c * 16 + i;
                            if (key > q0 + r) p0 = 0.f;
                            if (key + 1 > q0 + r) p1 = 0.f;
                        }
                        unpack_f32x2(fmul2(pack_f32x2(p0, p1), fadd2(pack_f32x2(__uint_as_float(dv[i]), __uint_as_float(dv[i + 1])), ndlt)), d0, d1);
                        ds[i >> 1] = pack_bf16(d0, d1);
                    }
                    tmem_st8(s_addr + c * 8, ds);            // over my own (already loaded) S columns
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(10 + t));
            }
            if (ok) {
                ok = mbar_wait(bar(12 + t), qn & 1, abort_flag, p.status, 621);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (ok) {
                ok = mbar_wait(bar(16), (u & 1) ^ 1, abort_flag, p.status, 623);    // the previous user's store has read the staging tile
                ok = __all_sync(0xffffffffu, ok);
            }
            if (!ok) break;
            tc_fence_after();
            uint8_t* stage = sm + L::kOut;
#pragma unroll 1
            for (int c = 0; c < DH / 64; ++c) {
                uint32_t w[32];
                tmem_ld32(o_addr + c * 32, w);
                tc_wait_ld();
                if (c == DH / 64 - 1) {                     // this thread's part of dQ_t has left TMEM
                    tc_fence_before();
                    mbar_arrive(bar(14 + t));
                }
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(w[8 * g + i]) * p.scale;
                    const int col = hf * (DH / 2) + c * 32 + g * 8, blk = col >> 6, chunk = (col & 63) >> 3;
                    *reinterpret_cast<uint4*>(stage + blk * 16384 + r * 128 + ((chunk ^ (r & 7)) << 4)) = pack8(f);
                }
            }
            fence_proxy_async();
            named_bar_sync(1 + t, 256);
            if (leader) {
                for (int kb = 0; kb < L::kBlocks; ++kb)
                    tma_store_2d(&tmOut, sbase + L::kOut + kb * 16384, it.h * DH + kb * 64, it.b * p.S + q0);
                bulk_commit();
                bulk_wait_read0();                          // the staging tile may be written again
                mbar_arrive(bar(16));
            }
            ++qn;
        }
        if (leader) bulk_wait0();
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
    p.B = B; p.tiles_per_seq = (S + 255) / 256; p.n_items = B * H * p.tiles_per_seq;
    p.sched = status->sched + 2;
    dim3 grid(p.n_items < rt->sm_count ? p.n_items : rt->sm_count);
    const cudaError_t e2 = dh == 64
        ? launch_k(attn_bwd_dq_tc_kernel<64>, grid, dim3(kDqThreads), DqSmem<64>::kBytes, stream, tmQ, tmDO, tmKV, tmOut, p)
        : launch_k(attn_bwd_dq_tc_kernel<128>, grid, dim3(kDqThreads), DqSmem<128>::kBytes, stream, tmQ, tmDO, tmKV, tmOut, p);
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
    p.B = B; p.tiles_per_seq = S / 128; p.n_items = B * H * p.tiles_per_seq;
    p.sched = status->sched + 4;
    dim3 grid(p.n_items < rt->sm_count ? p.n_items : rt->sm_count);
    const cudaError_t e2 = dh == 64
        ? launch_k(attn_bwd_dkdv_tc_kernel<64>, grid, dim3(kThreads), KvSmem<64>::kBytes, stream, tmKV, tmQ, tmDO, tmOut, p)
        : launch_k(attn_bwd_dkdv_tc_kernel<128>, grid, dim3(kThreads), KvSmem<128>::kBytes, stream, tmKV, tmQ, tmDO, tmOut, p);
    return e2 == cudaSuccess ? nullptr : "attention bwd (dk, dv) launch failed";
}

}  // namespace pw
