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

constexpr int kThreads = 320;
constexpr float kLog2e = 1.4426950408889634f;

template <int DH>
struct FwdSmem {
    static constexpr int kBlocks = DH / 64;                 // 64-column (128-byte) blocks per row
    static constexpr int kTile = 128 * DH * 2;              // one 128-row tile of Q, K or V
    static constexpr int kQ = 0;                            // two Q tiles
    static constexpr int kK = 2 * kTile;                    // two K stages
    static constexpr int kV = 4 * kTile;                    // two V stages
    static constexpr int kBars = 6 * kTile;
    static constexpr int kBytes = kBars + 256 + 1024;
};

struct FwdParams {
    int S, H;
    float scale;
    float* lse;
    DeviceStatus* status;
};

template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQKV, const __grid_constant__ CUtensorMap tmO, const FwdParams p)
{
    using L = FwdSmem<DH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(sm);
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
    // barrier map: 0 q_full | 1,2 k_full | 3,4 k_empty | 5,6 v_full | 7,8 v_empty | 9,10 s_full | 11,12 p_full | 13,14 o_full
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
    const int nA = q0A / 128 + 1, nB = hasB ? nA + 1 : 0;   // key tiles each query tile needs
    const int n_kv = hasB ? nB : nA;
    const int row_base = b * p.S;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 11; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(11), 128); mbar_init(bar(12), 128);
        mbar_init(bar(13), 1); mbar_init(bar(14), 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
        prefetch_tmap(&tmQKV);
        prefetch_tmap(&tmO);
    }
    grid_dep_launch();
    grid_dep_wait();                                        // qkv comes from the previous kernel
    if (threadIdx.x == 0) {
        // first loads go out before the TMEM allocation and the CTA-wide barrier
        const int nq = hasB ? 2 : 1;
        mbar_arrive_expect_tx(bar(0), nq * L::kTile);
        for (int t = 0; t < nq; ++t)
            for (int kb = 0; kb < L::kBlocks; ++kb)
                tma_load_2d(sbase + L::kQ + t * L::kTile + kb * 16384, &tmQKV, h * DH + kb * 64,
                            row_base + q0A + t * 128, bar(0));
        mbar_arrive_expect_tx(bar(1), L::kTile);
        mbar_arrive_expect_tx(bar(5), L::kTile);
        for (int kb = 0; kb < L::kBlocks; ++kb) {
            tma_load_2d(sbase + L::kK + kb * 16384, &tmQKV, d + h * DH + kb * 64, row_base, bar(1));
            tma_load_2d(sbase + L::kV + kb * 16384, &tmQKV, 2 * d + h * DH + kb * 64, row_base, bar(5));
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
            for (int j = 1; j < n_kv; ++j) {                // Q and key tile 0 were requested in the prologue
                const int s = j & 1, ph = (j >> 1) & 1;
                if (!mbar_wait(bar(3 + s), ph ^ 1, abort_flag, p.status, 400)) break;
                mbar_arrive_expect_tx(bar(1 + s), L::kTile);
                for (int kb = 0; kb < L::kBlocks; ++kb)
                    tma_load_2d(sbase + L::kK + s * L::kTile + kb * 16384, &tmQKV, d + h * DH + kb * 64,
                                row_base + j * 128, bar(1 + s));
                if (!mbar_wait(bar(7 + s), ph ^ 1, abort_flag, p.status, 401)) break;
                mbar_arrive_expect_tx(bar(5 + s), L::kTile);
                for (int kb = 0; kb < L::kBlocks; ++kb)
                    tma_load_2d(sbase + L::kV + s * L::kTile + kb * 16384, &tmQKV, 2 * d + h * DH + kb * 64,
                                row_base + j * 128, bar(5 + s));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, DH, false, true);
            // S_t = Q_t K^T from K stage s
            auto issue_s = [&](int t, int s) {
                const uint64_t dq = make_smem_desc_sw128(sbase + L::kQ + t * L::kTile, 16, 1024);
                const uint64_t dk = make_smem_desc_sw128(sbase + L::kK + s * L::kTile, 16, 1024);
                const uint32_t dst = tmem_base + t * 128;
#pragma unroll
                for (int kb = 0; kb < L::kBlocks; ++kb)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_f16(dst, desc_advance(dq, kb * 16384 + kk * 32), desc_advance(dk, kb * 16384 + kk * 32),
                                 idesc_s, (kb | kk) ? 1u : 0u);
                umma_commit(bar(9 + t));
            };
            // O_t (+)= P_t V from V stage s; P_t is bf16 packed in the first 64 columns of S_t
            auto issue_pv = [&](int t, int s, bool acc) {
                const uint64_t dv = make_smem_desc_sw128(sbase + L::kV + s * L::kTile, 16384, 1024);
                const uint32_t dst = tmem_base + 256 + t * 128, src = tmem_base + t * 128;
                umma_f16_ta(dst, src, dv, idesc_pv, acc ? 1u : 0u);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks)
                    umma_f16_ta(dst, src + ks * 8, desc_advance(dv, ks * 2048), idesc_pv, 1u);
            };
            bool ok = mbar_wait(bar(0), 0, abort_flag, p.status, 410) && mbar_wait(bar(1), 0, abort_flag, p.status, 411);
            if (ok) {
                tc_fence_after();
                issue_s(0, 0);
                if (hasB) issue_s(1, 0);
                umma_commit(bar(3));
            }
            for (int j = 0; j < n_kv && ok; ++j) {
                const int s = j & 1, ph = (j >> 1) & 1, nxt = j + 1, sn = nxt & 1, phn = (nxt >> 1) & 1;
                if (!mbar_wait(bar(5 + s), ph, abort_flag, p.status, 412)) { ok = false; break; }
                bool k_waited = false;
                if (j < nA) {
                    if (!mbar_wait(bar(11), j & 1, abort_flag, p.status, 413)) { ok = false; break; }
                    tc_fence_after();
                    issue_pv(0, s, j > 0);
                    if (j == nA - 1) umma_commit(bar(13));
                }
                if (nxt < nA) {
                    if (!mbar_wait(bar(1 + sn), phn, abort_flag, p.status, 414)) { ok = false; break; }
                    k_waited = true;
                    tc_fence_after();
                    issue_s(0, sn);
                }
                if (j < nB) {
                    if (!mbar_wait(bar(12), j & 1, abort_flag, p.status, 415)) { ok = false; break; }
                    tc_fence_after();
                    issue_pv(1, s, j > 0);
                    if (j == nB - 1) umma_commit(bar(14));
                }
                umma_commit(bar(7 + s));                    // V stage free once these MMAs are done
                if (nxt < nB) {
                    if (!k_waited && !mbar_wait(bar(1 + sn), phn, abort_flag, p.status, 416)) { ok = false; break; }
                    tc_fence_after();
                    issue_s(1, sn);
                }
                if (nxt < n_kv) umma_commit(bar(3 + sn));   // K stage free
            }
        }
    } else {
        const int t = (warp - 2) >> 2;                      // 0 = tile A, 1 = tile B
        const int q = warp & 3;                             // TMEM lane quarter this warp may touch
        const int r = q * 32 + lane;                        // query row inside the tile
        const int n_t = t == 0 ? nA : nB;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t s_addr = tmem_base + lane_addr + t * 128;
        const uint32_t o_addr = tmem_base + lane_addr + 256 + t * 128;
        const float sl2 = p.scale * kLog2e;
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_t; ++j) {
            ok = mbar_wait(bar(9 + t), j & 1, abort_flag, p.status, 420);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const bool diag = j == n_t - 1;
            // all 128 scores of the row in registers (four loads in flight, one wait)
            uint32_t v[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, v + c * 32);
            tc_wait_ld();
            // row maximum: eight independent chains of three-input max (64 instructions for 128 scores)
            float mxs[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) mxs[k] = -INFINITY;
            if (diag) {
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    if (i <= r) mxs[i & 7] = fmaxf(mxs[i & 7], __uint_as_float(v[i]));
            } else {
#pragma unroll
                for (int i = 0; i < 128; i += 2)
                    mxs[(i >> 1) & 7] = fmax3(mxs[(i >> 1) & 7], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
            }
            const float mx = fmaxf(fmax3(mxs[0], mxs[1], mxs[2]), fmax3(fmaxf(mxs[3], mxs[4]), fmaxf(mxs[5], mxs[6]), mxs[7]));
            const float m_new = fmaxf(m_used, mx);
            const bool grow = (m_new - m_used) * sl2 > 8.0f;        // also true on the first tile (m_used = -inf)
            if (j == 0) {
                m_used = m_new;
            } else if (__any_sync(0xffffffffu, grow)) {
                const float alpha = grow ? ex2_approx((m_used - m_new) * sl2) : 1.0f;
                if (grow) m_used = m_new;
                l *= alpha;
#pragma unroll 1
                for (int c = 0; c < DH / 32; ++c) {
                    uint32_t w[32];
                    tmem_ld32(o_addr + c * 32, w);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(__uint_as_float(w[i]) * alpha);
                    tmem_st32(o_addr + c * 32, w);
                }
            }
            // p = exp2((s - m) * scale * log2e), packed bf16 written over the S columns
            const float mb = m_used * sl2;
            if (diag) {
                float ls = 0.f;
#pragma unroll
                for (int i = 0; i < 128; i += 2) {
                    float p0 = i > r ? 0.f : ex2_approx(fmaf(__uint_as_float(v[i]), sl2, -mb));
                    float p1 = i + 1 > r ? 0.f : ex2_approx(fmaf(__uint_as_float(v[i + 1]), sl2, -mb));
                    ls += p0 + p1;
                    v[i >> 1] = pack_bf16(p0, p1);
                }
                l += ls;
            } else {
                // two scores per FMA / add instruction; the exponentials stay on the MUFU
                const uint64_t sl2x2 = pack_f32x2(sl2, sl2), mbx2 = pack_f32x2(-mb, -mb);
                uint64_t lsum[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int i = 0; i < 128; i += 2) {
                    float a0, a1;
                    unpack_f32x2(ffma2(pack_f32x2(__uint_as_float(v[i]), __uint_as_float(v[i + 1])), sl2x2, mbx2), a0, a1);
                    const float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                    lsum[(i >> 1) & 3] = fadd2(lsum[(i >> 1) & 3], pack_f32x2(p0, p1));
                    v[i >> 1] = pack_bf16(p0, p1);
                }
                float s0, s1;
                unpack_f32x2(fadd2(fadd2(lsum[0], lsum[1]), fadd2(lsum[2], lsum[3])), s0, s1);
                l += s0 + s1;
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_st16(s_addr + c * 16, v + c * 16);
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar(11 + t));
        }
        if (ok && n_t > 0) {
            ok = mbar_wait(bar(13 + t), 0, abort_flag, p.status, 421);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok && n_t > 0) {
            tc_fence_after();
            const float inv_l = 1.0f / l;
            uint8_t* stage = sm + L::kQ + t * L::kTile;     // the Q tile is idle now: reuse it for O
#pragma unroll 1
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(o_addr + c * 32, v);
                tc_wait_ld();
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * g + i]) * inv_l;
                    const int col = c * 32 + g * 8, blk = col >> 6, chunk = (col & 63) >> 3;
                    *reinterpret_cast<uint4*>(stage + blk * 16384 + r * 128 + ((chunk ^ (r & 7)) << 4)) = pack8(f);
                }
            }
            p.lse[(static_cast<size_t>(b) * p.H + h) * p.S + (t == 0 ? q0A : q0B) + r] = m_used * p.scale + logf(l);
            fence_proxy_async();
            named_bar_sync(1 + t, 128);
            if ((warp & 3) == 2 && lane == 0) {
                for (int kb = 0; kb < L::kBlocks; ++kb)
                    tma_store_2d(&tmO, sbase + L::kQ + t * L::kTile + kb * 16384, h * DH + kb * 64,
                                 row_base + (t == 0 ? q0A : q0B));
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
    p.S = S; p.H = H; p.scale = 1.0f / sqrtf(static_cast<float>(dh));
    p.lse = static_cast<float*>(lse);
    p.status = status;
    dim3 grid((S + 255) / 256, B * H);
    const cudaError_t e2 = dh == 64
        ? launch_k(attn_fwd_tc_kernel<64>, grid, dim3(kThreads), FwdSmem<64>::kBytes, stream, tmQKV, tmO, p)
        : launch_k(attn_fwd_tc_kernel<128>, grid, dim3(kThreads), FwdSmem<128>::kBytes, stream, tmQKV, tmO, p);
    return e2 == cudaSuccess ? nullptr : "attention fwd launch failed";
}

}  // namespace pw
