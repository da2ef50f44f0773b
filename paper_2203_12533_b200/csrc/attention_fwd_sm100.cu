// Causal attention forward on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// One CTA owns two adjacent 128-query tiles (A, B) of one (sequence, head) and streams the
// 128-key tiles up to the diagonal through a 2-stage K ring and a 2-stage V ring.  10 warps:
//   warp 0      TMA producer (one lane): Q once, then K_j / V_j.
//   warp 1      MMA issuer (one lane), owns the TMEM allocation (512 columns):
//                 S_t = Q_t K_j^T   (128x128, fp32)  -> columns t*128
//                 O_t += P_t V_j    (128xdh,  fp32)  -> columns 256 + t*128, P_t read from TMEM
//               issued so that the tensor pipe works on one tile while the other is in softmax:
//               PV_A(j), S_A(j+1), PV_B(j), S_B(j+1), ...
//   warps 2..5  softmax of tile A, warps 6..9 softmax of tile B (thread = one query row = one TMEM
//               lane): row max, exp2 with the 1/sqrt(dh) scale folded in, row sum, P written back
//               as packed bf16 over the S columns it came from.  The running maximum is only
//               advanced when it grows by more than 8 (in log2 units); only then is O rescaled in
//               TMEM (tcgen05.ld / st) - P stays below 2^8, exact after the final division by l.
// The epilogue divides O by l, stages it as bf16 in the (now idle) Q tile and stores it with TMA.
// Every mbarrier wait is bounded; on expiry all roles leave, TMEM is released, the status word
// records PW_ERR_TIMEOUT.
#include "pw_kernels.h"

namespace pw {
namespace {

constexpr int kThreads = 576;                              // producer warp, MMA warp, 2 x 8 softmax warps
constexpr float kLog2e = 1.4426950408889634f;

template <int DH>
struct FwdSmem {
    static constexpr int kBlocks = DH / 64;                 // 64-column (128-byte) blocks per row
    static constexpr int kTile = 128 * DH * 2;              // one 128-row tile of Q, K or V
    static constexpr int kQ = 0;                            // two Q tiles
    static constexpr int kK = 2 * kTile;                    // two K stages
    static constexpr int kV = 4 * kTile;                    // two V stages
    static constexpr int kO = 6 * kTile;                    // output staging tile (shared by both query tiles)
    static constexpr int kBars = 7 * kTile;
    static constexpr int kXch = kBars + 256;                // per-row exchange between the two threads of a row: [tile][half][128] fp32
    static constexpr int kEnd = kXch + 2 * 2 * 128 * 4;
    static constexpr int kBytes = kEnd + ((kEnd + 1024 <= 232448) ? 1024 : 232448 - kEnd);   // alignment slack (checked in the kernel)
};


struct FwdParams {
    int S, H, B;
    int pairs_per_seq;          // ceil(S / 256)
    int n_items;                // B * H * pairs_per_seq
    float scale;
    float* lse;
    DeviceStatus* status;
    int* sched;                 // {next ticket, CTAs done}
};

// Work items (one per sequence, head and pair of query tiles) are numbered heaviest first (latest
// query tiles first) and handed out in that order: the producer thread draws the next number from
// a global counter and passes it to the other roles through a two-slot ring in shared memory, so
// the causal triangle balances itself over the CTAs.  Every CTA draws exactly one number past the
// end; the last CTA to do so clears the counters for the next launch.
struct FwdItem { int b, h, q0A, nA, nB; };
__device__ __forceinline__ bool fwd_item(const FwdParams& p, int idx, FwdItem& it)
{
    if (idx >= p.n_items) return false;
    const int BH = p.B * p.H;
    const int pair = p.pairs_per_seq - 1 - idx / BH, bh = idx % BH;
    it.b = bh / p.H; it.h = bh % p.H;
    it.q0A = pair * 256;
    it.nA = it.q0A / 128 + 1;                               // key tiles each query tile needs
    it.nB = it.q0A + 128 < p.S ? it.nA + 1 : 0;
    return true;
}

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQKV, const __grid_constant__ CUtensorMap tmO, const FwdParams p)
{
    using L = FwdSmem<DH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(sm);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
    // barrier map (t = query tile, s = ring stage):
    //   0+t q_full | 2+t q_empty | 4+s k_full | 6+s k_empty | 8+s v_full | 10+s v_empty
    //   12+t s_full | 14+t p_full (128 arrivals) | 16+t o_full | 18+t o_empty (128 arrivals) | 20 staging free
    //   21+i item_full | 23+i item_empty (17 arrivals: MMA warp + 16 softmax warps)
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
    volatile int* item_slot = reinterpret_cast<volatile int*>(tmem_slot + 2);   // two entries
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
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
    if (sm + L::kEnd > smem_raw + L::kBytes) {              // the alignment ate more than the slack (never seen; fail loudly)
        if (threadIdx.x == 0 && atomicCAS(&p.status->code, 0, kStatusTimeout) == 0) p.status->site = 499;
        return;
    }

    auto load_q = [&](const FwdItem& it, int t) {
        mbar_arrive_expect_tx(bar(0 + t), L::kTile);
        for (int kb = 0; kb < L::kBlocks; ++kb)
            tma_load_2d(sbase + L::kQ + t * L::kTile + kb * 16384, &tmQKV, it.h * DH + kb * 64,
                        it.b * p.S + it.q0A + t * 128, bar(0 + t));
    };
    auto load_k = [&](const FwdItem& it, int j, int s) {
        mbar_arrive_expect_tx(bar(4 + s), L::kTile);
        for (int kb = 0; kb < L::kBlocks; ++kb)
            tma_load_2d(sbase + L::kK + s * L::kTile + kb * 16384, &tmQKV, d + it.h * DH + kb * 64,
                        it.b * p.S + j * 128, bar(4 + s));
    };
    auto load_v = [&](const FwdItem& it, int j, int s) {
        mbar_arrive_expect_tx(bar(8 + s), L::kTile);
        for (int kb = 0; kb < L::kBlocks; ++kb)
            tma_load_2d(sbase + L::kV + s * L::kTile + kb * 16384, &tmQKV, 2 * d + it.h * DH + kb * 64,
                        it.b * p.S + j * 128, bar(8 + s));
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < 14; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(14), 256); mbar_init(bar(15), 256);
        mbar_init(bar(16), 1); mbar_init(bar(17), 1);
        mbar_init(bar(18), 256); mbar_init(bar(19), 256);
        mbar_init(bar(20), 1);
        mbar_init(bar(21), 1); mbar_init(bar(22), 1);
        mbar_init(bar(23), 17); mbar_init(bar(24), 17);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmQKV);
        prefetch_tmap(&tmO);
    }
    grid_dep_launch();
    grid_dep_wait();                                        // qkv comes from the previous kernel
    if (threadIdx.x == 0) {
        // the first item's first loads go out before the TMEM allocation and the CTA-wide barrier
        FwdItem it;
        const int idx0 = draw();
        item_slot[0] = idx0;
        mbar_arrive(bar(21));
        if (fwd_item(p, idx0, it)) {
            load_k(it, 0, 0);
            load_q(it, 0);
            if (it.nB) load_q(it, 1);
            load_v(it, 0, 0);
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
            uint32_t n = 0;                                 // key/value tiles requested so far
            uint32_t qn[2] = {0, 0};                        // items each query tile took part in
            bool ok = true;
            FwdItem it;
            int idx = item_slot[0];
            for (int k = 0; ok && fwd_item(p, idx, it); ++k) {
                const int n_kv = it.nB ? it.nB : it.nA;
                for (int j = 0; j < n_kv && ok; ++j, ++n) {
                    const int s = n & 1;
                    const uint32_t ph = (n >> 1) & 1;
                    const bool early = k == 0 && j == 0;    // requested in the prologue
                    if (!early) {
                        if (!mbar_wait(bar(6 + s), ph ^ 1, abort_flag, p.status, 400)) { ok = false; break; }
                        load_k(it, j, s);
                    }
                    if (j == 0) {
                        // Q follows the first key tile; its buffer is free once the previous item's
                        // last S = Q K^T has been computed.
                        for (int t = 0; t < (it.nB ? 2 : 1) && ok; ++t) {
                            if (!early) {
                                if (!mbar_wait(bar(2 + t), (qn[t] & 1) ^ 1, abort_flag, p.status, 402)) { ok = false; break; }
                                load_q(it, t);
                            }
                            ++qn[t];
                        }
                        if (!ok) break;
                    }
                    if (!early) {
                        if (!mbar_wait(bar(10 + s), ph ^ 1, abort_flag, p.status, 401)) { ok = false; break; }
                        load_v(it, j, s);
                    }
                }
                if (!ok) break;
                // next item: its number goes into slot (k+1)&1 once every role has read what was there
                const int kn = k + 1;
                if (!mbar_wait(bar(23 + (kn & 1)), ((kn >> 1) & 1) ^ 1, abort_flag, p.status, 403)) break;
                idx = draw();
                item_slot[kn & 1] = idx;
                mbar_arrive(bar(21 + (kn & 1)));
            }
        }
    } else if (warp == 1) {
        // The whole warp runs this role converged (waits and address arithmetic stay uniform);
        // one elected lane issues the tcgen05 instructions.
        constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);
        constexpr uint32_t idesc_pv = make_idesc_bf16(128, DH, false, true);
        const uint32_t tb = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t sb = __shfl_sync(0xffffffffu, sbase, 0);
        // S_t = Q_t K^T from K stage s
        auto issue_s = [&](int t, int s) {
            const uint64_t dq = make_smem_desc_sw128(sb + L::kQ + t * L::kTile, 16, 1024);
            const uint64_t dk = make_smem_desc_sw128(sb + L::kK + s * L::kTile, 16, 1024);
            const uint32_t dst = tb + t * 128;
            if (elect_one()) {
#pragma unroll
                for (int kb = 0; kb < L::kBlocks; ++kb)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_f16(dst, desc_advance(dq, kb * 16384 + kk * 32), desc_advance(dk, kb * 16384 + kk * 32),
                                 idesc_s, (kb | kk) ? 1u : 0u);
                umma_commit(bar(12 + t));
            }
            __syncwarp();
        };
        // O_t (+)= P_t V from V stage s; P_t is bf16 packed over the S columns it came from: the 16
        // keys of step ks sit in 8 columns at (ks/4)*64 + ((ks%4)/2)*32 + (ks%2)*8 of S_t
        auto issue_pv = [&](int t, int s, bool acc) {
            const uint64_t dv = make_smem_desc_sw128(sb + L::kV + s * L::kTile, 16384, 1024);
            const uint32_t dst = tb + 256 + t * 128, src = tb + t * 128;
            if (elect_one()) {
                umma_f16_ta(dst, src, dv, idesc_pv, acc ? 1u : 0u);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks)
                    umma_f16_ta(dst, src + (ks >> 2) * 64 + ((ks & 3) >> 1) * 32 + (ks & 1) * 8, desc_advance(dv, ks * 2048), idesc_pv, 1u);
            }
            __syncwarp();
        };
        auto commit = [&](int b) {
            if (elect_one()) umma_commit(bar(b));
            __syncwarp();
        };
        auto wait = [&](int b, uint32_t parity, int site) {
            bool w = mbar_wait(bar(b), parity, abort_flag, p.status, site);
            return __all_sync(0xffffffffu, w);
        };
        uint32_t n = 0;                                 // key/value tiles consumed before this item
        uint32_t np[2] = {0, 0};                        // P tiles consumed per query tile
        uint32_t qn[2] = {0, 0};                        // items each query tile took part in
        bool ok = true;
        FwdItem it;
        for (int k = 0; ok; ++k) {
            if (!wait(21 + (k & 1), (k >> 1) & 1, 423)) break;
            const int idx = __shfl_sync(0xffffffffu, item_slot[k & 1], 0);   // broadcast: everything derived from it is warp-uniform
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(23 + (k & 1)));
            if (!fwd_item(p, idx, it)) break;
            const int nA = it.nA, nB = it.nB, n_kv = nB ? nB : nA;
            {
                const int s = n & 1;
                const uint32_t ph = (n >> 1) & 1;
                ok = wait(4 + s, ph, 411) && wait(0, qn[0] & 1, 410);
                if (!ok) break;
                tc_fence_after();
                issue_s(0, s);
                if (nA == 1) commit(2);                     // Q_A is not needed again
                if (nB) {
                    if (!wait(1, qn[1] & 1, 417)) { ok = false; break; }
                    tc_fence_after();
                    issue_s(1, s);
                    if (nB == 1) commit(3);
                }
                commit(6 + s);
            }
            for (int j = 0; j < n_kv && ok; ++j) {
                const uint32_t nj = n + j, nn = nj + 1;
                const int s = nj & 1, sn = nn & 1;
                const uint32_t ph = (nj >> 1) & 1, phn = (nn >> 1) & 1;
                if (!wait(8 + s, ph, 412)) { ok = false; break; }
                bool k_waited = false;
                if (j < nA) {
                    if (!wait(14, np[0] & 1, 413)) { ok = false; break; }
                    ++np[0];
                    // the previous item's O_A must have been read out before it is overwritten
                    if (j == 0 && !wait(18, (qn[0] & 1) ^ 1, 418)) { ok = false; break; }
                    tc_fence_after();
                    issue_pv(0, s, j > 0);
                    if (j == nA - 1) commit(16);
                }
                if (j + 1 < nA) {
                    if (!wait(4 + sn, phn, 414)) { ok = false; break; }
                    k_waited = true;
                    tc_fence_after();
                    issue_s(0, sn);
                    if (j + 2 == nA) commit(2);
                }
                if (j < nB) {
                    if (!wait(15, np[1] & 1, 415)) { ok = false; break; }
                    ++np[1];
                    if (j == 0 && !wait(19, (qn[1] & 1) ^ 1, 419)) { ok = false; break; }
                    tc_fence_after();
                    issue_pv(1, s, j > 0);
                    if (j == nB - 1) commit(17);
                }
                commit(10 + s);                             // V stage free once these MMAs are done
                if (j + 1 < nB) {
                    if (!k_waited && !wait(4 + sn, phn, 416)) { ok = false; break; }
                    tc_fence_after();
                    issue_s(1, sn);
                    if (j + 2 == nB) commit(3);
                }
                if (j + 1 < n_kv) commit(6 + sn);           // K stage free
            }
            n += n_kv;
            ++qn[0];
            if (nB) ++qn[1];
        }
    } else {
        // Softmax: two threads per query row.  Warps 2..9 serve tile A, 10..17 tile B; inside a tile
        // the warp's TMEM lane quarter is warp % 4 and its column half hf is (warp - 2) / 4 % 2: a
        // thread owns 64 of the row's 128 scores (P goes back over the first 32 of their columns) and half of the
        // O columns.  The two threads of a row swap their partial row maxima (and, at the end, row
        // sums) through shared memory under a 256-thread named barrier - that barrier also orders
        // every thread's S loads before any P store (P overwrites the S columns).
        const int t = (warp - 2) >> 3;                      // 0 = tile A, 1 = tile B
        const int hf = ((warp - 2) >> 2) & 1;               // column half
        const int q = warp & 3;                             // TMEM lane quarter this warp may touch
        const int r = q * 32 + lane;                        // query row inside the tile
        const bool leader = hf == 0 && q == 2 && lane == 0;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t s_addr = tmem_base + lane_addr + t * 128 + hf * 64;       // my 64 scores
        const uint32_t o_addr = tmem_base + lane_addr + 256 + t * 128 + hf * (DH / 2);
        float* xch = reinterpret_cast<float*>(sm + L::kXch) + t * 256;           // [half][row]
        const float sl2 = p.scale * kLog2e;
        uint32_t ns = 0, qn = 0;                            // S tiles and items this query tile has seen
        uint32_t u_base = 0;                                // uses of the output staging tile before this item
        bool ok = true;
        FwdItem it;
        for (int k = 0; ok; ++k) {
        ok = mbar_wait(bar(21 + (k & 1)), (k >> 1) & 1, abort_flag, p.status, 424);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const int idx = item_slot[k & 1];
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(23 + (k & 1)));
        if (!fwd_item(p, idx, it)) break;
        const int n_t = t == 0 ? it.nA : it.nB;
        const uint32_t u = u_base + t;                      // staging order: A(k), B(k), A(k+1), ...
        u_base += it.nB ? 2 : 1;
        if (n_t == 0) continue;
        const int q0 = it.q0A + t * 128;
        float m_used = -INFINITY, l = 0.f;
        for (int j = 0; j < n_t; ++j, ++ns) {
            ok = mbar_wait(bar(12 + t), ns & 1, abort_flag, p.status, 420);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const bool diag = j == n_t - 1;
            const int lim = diag ? r - hf * 64 : 64;        // columns i > lim of my 64 are masked (diagonal tile)
            // pass 1: row maximum.  Scores 0..31 are read, used and dropped; scores 32..63 stay in
            // registers for the second pass (all 64 would not fit under the 576-thread register limit).
            float mxs[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            uint32_t vk[32];
            {
                uint32_t v[32];
                tmem_ld32(s_addr, v);
                tmem_ld32(s_addr + 32, vk);
                tc_wait_ld();
                if (diag) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        v[i] = i > lim ? 0xff800000u : v[i];
                        vk[i] = 32 + i > lim ? 0xff800000u : vk[i];
                    }
                }
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    mxs[(i >> 1) & 1] = fmax3(mxs[(i >> 1) & 1], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                    mxs[2 + ((i >> 1) & 1)] = fmax3(mxs[2 + ((i >> 1) & 1)], __uint_as_float(vk[i]), __uint_as_float(vk[i + 1]));
                }
            }
            const float mine = fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3]));
            xch[hf * 128 + r] = mine;
            named_bar_sync(1 + t, 256);
            const float mx = fmaxf(mine, xch[(hf ^ 1) * 128 + r]);
            const float m_new = fmaxf(m_used, mx);
            const bool grow = (m_new - m_used) * sl2 > 8.0f;        // also true on the first tile (m_used = -inf)
            if (j == 0) {
                m_used = m_new;
            } else if (__any_sync(0xffffffffu, grow)) {     // both threads of a row see the same values
                const float alpha = grow ? ex2_approx((m_used - m_new) * sl2) : 1.0f;
                if (grow) m_used = m_new;
                l *= alpha;
#pragma unroll 1
                for (int c = 0; c < DH / 64; ++c) {
                    uint32_t w[32];
                    tmem_ld32(o_addr + c * 32, w);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(__uint_as_float(w[i]) * alpha);
                    tmem_st32(o_addr + c * 32, w);
                }
            }
            // pass 2: p = exp2((s - m) * scale * log2e), packed bf16 written over my own S columns: first the
            // kept scores 32..63 (into columns 32..47, their own), then scores 0..31 re-read (into columns 0..15)
            const float mb = m_used * sl2;
            const uint64_t sl2x2 = pack_f32x2(sl2, sl2), mbx2 = pack_f32x2(-mb, -mb);
            uint64_t lsum[2] = {0ull, 0ull};
            auto exps = [&](uint32_t* v) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    // the MUFU bounds this loop: every fourth pair takes the FMA-pipe exponential
                    const uint64_t a = ffma2(pack_f32x2(__uint_as_float(v[i]), __uint_as_float(v[i + 1])), sl2x2, mbx2);
                    uint64_t pe;
                    if (((i >> 1) & 3) == 3) {
                        pe = exp2_poly2(a);
                    } else {
                        float a0, a1;
                        unpack_f32x2(a, a0, a1);
                        pe = pack_f32x2(ex2_approx(a0), ex2_approx(a1));
                    }
                    lsum[(i >> 1) & 1] = fadd2(lsum[(i >> 1) & 1], pe);
                    float p0, p1;
                    unpack_f32x2(pe, p0, p1);
                    v[i >> 1] = pack_bf16(p0, p1);
                }
            };
            {
                uint32_t v[32];
                tmem_ld32(s_addr, v);                        // in flight while the kept half is processed
                exps(vk);
                tmem_st16(s_addr + 32, vk);
                tc_wait_ld();
                if (diag) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = i > lim ? 0xff800000u : v[i];
                }
                exps(v);
                tmem_st16(s_addr, v);
            }
            {
                float s0, s1;
                unpack_f32x2(fadd2(lsum[0], lsum[1]), s0, s1);
                l += s0 + s1;
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar(14 + t));
        }
        if (ok) {
            ok = mbar_wait(bar(16 + t), qn & 1, abort_flag, p.status, 421);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (!ok) break;
        {
            tc_fence_after();
            // row sum = the two halves' sums (the partner's last read of this slot was before its last p_full arrival)
            xch[hf * 128 + r] = l;
            named_bar_sync(1 + t, 256);
            const float l_row = l + xch[(hf ^ 1) * 128 + r];
            const float inv_l = 1.0f / l_row;
            uint8_t* stage = sm + L::kO;
            ok = mbar_wait(bar(20), (u & 1) ^ 1, abort_flag, p.status, 422);    // the previous user's store has read it
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
#pragma unroll 1
            for (int c = 0; c < DH / 64; ++c) {
                uint32_t w[32];
                tmem_ld32(o_addr + c * 32, w);
                tc_wait_ld();
                if (c == DH / 64 - 1) {                     // this thread's part of O_t has left TMEM
                    tc_fence_before();
                    mbar_arrive(bar(18 + t));
                }
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(w[8 * g + i]) * inv_l;
                    const int col = hf * (DH / 2) + c * 32 + g * 8, blk = col >> 6, chunk = (col & 63) >> 3;
                    *reinterpret_cast<uint4*>(stage + blk * 16384 + r * 128 + ((chunk ^ (r & 7)) << 4)) = pack8(f);
                }
            }
            if (hf == 0) p.lse[(static_cast<size_t>(it.b) * p.H + it.h) * p.S + q0 + r] = m_used * p.scale + logf(l_row);
            fence_proxy_async();
            named_bar_sync(1 + t, 256);
            if (leader) {
                for (int kb = 0; kb < L::kBlocks; ++kb)
                    tma_store_2d(&tmO, sbase + L::kO + kb * 16384, it.h * DH + kb * 64, it.b * p.S + q0);
                bulk_commit();
                bulk_wait_read0();                          // the staging tile may be written again
                mbar_arrive(bar(20));
            }
            ++qn;
        }
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

// bf16 [rows, cols] row-major, box 64 columns x 128 rows, 128-byte swizzle.
const char* encode_rows(Runtime* rt, CUtensorMap* map, const void* ptr, uint64_t cols, uint64_t rows)
{
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(rt->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? nullptr : "cuTensorMapEncodeTiled failed";
}

}  // namespace


const char* configure_attention_fwd()
{
    if (cudaFuncSetAttribute(attn_fwd_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<64>::kBytes) != cudaSuccess ||
        cudaFuncSetAttribute(attn_fwd_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<128>::kBytes) != cudaSuccess)
        return "cudaFuncSetAttribute(attention fwd) failed";
    return nullptr;
}

const char* launch_attention_fwd(Runtime* rt, const void* qkv, int B, int S, int H, int dh, void* o, void* lse,
                                 DeviceStatus* status, cudaStream_t stream)
{
    if (B <= 0 || H <= 0 || S <= 0 || (S % 128) != 0 || (dh != 64 && dh != 128)) return "attention: unsupported shape";
    const int d = H * dh;
    CUtensorMap tmQKV, tmO;
    const char* e;
    if ((e = encode_rows(rt, &tmQKV, qkv, 3ull * d, static_cast<uint64_t>(B) * S))) return e;
    if ((e = encode_rows(rt, &tmO, o, d, static_cast<uint64_t>(B) * S))) return e;
    FwdParams p;
    p.S = S; p.H = H; p.B = B; p.scale = 1.0f / sqrtf(static_cast<float>(dh));
    p.pairs_per_seq = (S + 255) / 256;
    p.n_items = B * H * p.pairs_per_seq;
    p.lse = static_cast<float*>(lse);
    p.status = status;
    p.sched = status->sched + 0;
    dim3 grid(p.n_items < rt->sm_count ? p.n_items : rt->sm_count);
    const cudaError_t e2 = dh == 64
        ? launch_k(attn_fwd_tc_kernel<64>, grid, dim3(kThreads), FwdSmem<64>::kBytes, stream, tmQKV, tmO, p)
        : launch_k(attn_fwd_tc_kernel<128>, grid, dim3(kThreads), FwdSmem<128>::kBytes, stream, tmQKV, tmO, p);
    return e2 == cudaSuccess ? nullptr : "attention fwd launch failed";
}

}  // namespace pw
