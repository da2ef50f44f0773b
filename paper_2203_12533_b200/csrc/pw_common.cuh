// Shared device helpers for the sm_100a kernels: bf16 packing, mbarrier / TMA / tcgen05 PTX
// wrappers, bounded waits with a device status word.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pw {

// Device status block owned by the runtime (one per handle): word 0 = status code
// (0 = ok), word 1 = site id of the wait that gave up.
// Words 2.. are the work counters of the persistent attention kernels: {next ticket, CTAs done}
// per kernel.  They are zero between launches (the last CTA of a launch clears its pair).
// A GEMM whose last round of tiles would leave at least half of the CTA pairs idle cuts each of those
// tiles in two along K; the two halves meet through a ticket per (tile, CTA of the pair, epilogue warp).
constexpr int kSplitMaxTiles = 40;                       // at most half of the CTA pairs' worth of tiles is cut
constexpr int kSplitTickets = kSplitMaxTiles * 2 * 16;
struct DeviceStatus {
    int code;
    int site;
    int sched[6];               // [0,1] attention fwd, [2,3] dQ, [4,5] dK/dV
    int tickets[kSplitTickets]; // split-K hand-off of the GEMM; always back to zero when a kernel ends normally
};

constexpr int kStatusTimeout = 6;  // == PW_ERR_TIMEOUT

// ---------------------------------------------------------------- bf16 helpers
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ void unpack8(const uint4& v, float* f)
{
    f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
    f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
}
__device__ __forceinline__ uint4 pack8(const float* f)
{
    uint4 v;
    v.x = pack_bf16(f[0], f[1]); v.y = pack_bf16(f[2], f[3]);
    v.z = pack_bf16(f[4], f[5]); v.w = pack_bf16(f[6], f[7]);
    return v;
}

// GeLU and its derivative in fp32.  The erf form uses the rational/exponential approximation
// erfc(x) ~ (a1 t + ... + a5 t^5) exp(-x^2), t = 1/(1 + p x), x >= 0 (absolute error about 2e-7,
// far below bf16 resolution); the exponential exp(-u^2/2) is shared with the density term of the
// derivative.  act == 1 selects the tanh form.
__device__ __forceinline__ void normal_cdf_pdf(float u, float& cdf, float& e /* exp(-u^2/2) */)
{
    const float ax = fabsf(u) * 0.7071067811865476f;
    const float t = __frcp_rn(fmaf(0.3275911f, ax, 1.0f));
    e = __expf(-ax * ax);
    float poly = fmaf(t, 1.061405429f, -1.453152027f);
    poly = fmaf(t, poly, 1.421413741f);
    poly = fmaf(t, poly, -0.284496736f);
    poly = fmaf(t, poly, 0.254829592f);
    const float half_tail = 0.5f * poly * t * e;      // = erfc(|u|/sqrt2) / 2
    cdf = u < 0.f ? half_tail : 1.0f - half_tail;
}
__device__ __forceinline__ float fast_tanh(float z)
{
    const float e2 = __expf(2.0f * z);
    return 1.0f - __fdividef(2.0f, e2 + 1.0f);
}
__device__ __forceinline__ float gelu_f(float u, int act)
{
    if (act == 1) {
        const float z = 0.7978845608028654f * (u + 0.044715f * u * u * u);
        return 0.5f * u * (1.0f + fast_tanh(z));
    }
    float cdf, e;
    normal_cdf_pdf(u, cdf, e);
    return u * cdf;
}
__device__ __forceinline__ float gelu_grad_f(float u, int act)
{
    if (act == 1) {
        const float z = 0.7978845608028654f * (u + 0.044715f * u * u * u);
        const float th = fast_tanh(z);
        const float dz = 0.7978845608028654f * (1.0f + 0.134145f * u * u);
        return 0.5f * (1.0f + th) + 0.5f * u * (1.0f - th * th) * dz;
    }
    float cdf, e;
    normal_cdf_pdf(u, cdf, e);
    return fmaf(u * 0.3989422804014327f, e, cdf);
}

// ---------------------------------------------------------------- programmatic dependent launch
// A kernel launched with the programmatic-serialization attribute may start while the previous
// kernel of its stream is still running.  grid_dep_launch() lets the next kernel be scheduled as
// early as possible; grid_dep_wait() blocks until the previous kernel has completed and its
// memory is visible - every kernel calls it before its first global-memory access, so only the
// launch latency and the on-chip set-up overlap.  Both are no-ops for a plain launch.
// Consequence for every kernel here: no input pointer is `const __restrict__` and nothing is read
// with __ldg - the compiler treats such loads as invariant over the kernel's lifetime and may hoist
// them above the wait, where the producer has not written the data yet.
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- shared-memory addresses
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, P;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Spins on try_wait; gives up after kWaitCycles SM cycles (about a second) or as
// soon as another thread of the CTA has raised `abort_flag`.  On expiry it records
// (kStatusTimeout, site) in the device status block and raises the flag.  Returns false when
// the caller must stop using the pipeline and head for its teardown.
constexpr long long kWaitCycles = 1ll << 31;

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStatus* status, int site, long long limit = kWaitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3ffu) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit) {
                *abort_flag = 1;
                if (status != nullptr && atomicCAS(&status->code, 0, kStatusTimeout) == 0) status->site = site;
                return false;
            }
        }
    }
    return true;
}

// One lane of the (converged) warp is picked; the rest of the warp's code stays uniform.
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "selp.b32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// ---------------------------------------------------------------- TMA (tiled, no cluster qualifiers)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// Shared -> global tiled store / fp32 reduce-add (out-of-range parts of the box are clipped).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int x, int y)
{
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// All of this thread's bulk groups have finished READING shared memory (it may be rewritten).
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// At most the newest of this thread's bulk groups may still be reading shared memory.
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// All of this thread's bulk groups are complete.
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// ---------------------------------------------------------------- tcgen05 / TMEM
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem desc] * B[smem desc]; bf16 inputs, fp32 accumulate, one CTA.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier gets one arrival when every tcgen05 operation this thread issued so far is done.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets lane (base+i), columns c..c+31.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// Same with the A operand read from tensor memory (bf16 pairs packed in 32-bit columns).
__device__ __forceinline__ void umma_f16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 16 consecutive columns.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Stores: thread i of the warp writes lane (base+i), 16 / 32 consecutive 32-bit columns.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Three-input maximum and two-wide fp32 FMA / add (one instruction for two lanes of work).
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Barrier among `count` threads of the CTA (ids 1..15; id 0 is __syncthreads).
__device__ __forceinline__ void named_bar_sync(int id, int count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// ---------------------------------------------------------------- CTA pairs (cta_group::2)
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose completion bytes are credited to a barrier that
// may live in the peer CTA of the pair (cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// One MMA over the pair: M = 256 (128 rows from each CTA's A tile), B halves from both CTAs.
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                              uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives on the barrier at this shared-memory offset in every CTA of `mask` once all MMAs issued
// so far by this thread are complete (this is a barrier signal, not a data copy).
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t mask)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}

// Shared-memory matrix descriptor for tcgen05.mma, 128-byte swizzle.
//   bits [0,14)  start address >> 4        bits [16,30) leading-dimension byte offset >> 4
//   bits [32,46) stride byte offset >> 4   bits [46,48) descriptor version (1 on sm_100)
//   bits [61,64) layout type (2 = 128-byte swizzle)
__device__ __forceinline__ uint64_t make_smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3ffffu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// Descriptor of the same operand starting `bytes` further on (bytes a multiple of 16, the new
// start still inside the 256 KB shared-memory window, so the add never carries out of the
// address field).  Lets the MMA-issuing thread build a descriptor once and step it with one add.
__device__ __forceinline__ uint64_t desc_advance(uint64_t d, uint32_t bytes) { return d + (bytes >> 4); }

// Instruction descriptor for kind::f16 with bf16 A/B and fp32 D.
//   [4,6) D format (1 = f32)  [7,10) A format (1 = bf16)  [10,13) B format (1 = bf16)
//   bit 15 A major (1 = MN-major)  bit 16 B major  [17,23) N >> 3  [24,29) M >> 4
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N, bool a_mn_major, bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

// 2^a for two values on the FMA / ALU pipes (no MUFU): a = n + f with n = round(a), f in [-0.5, 0.5];
// 2^f by a cubic (relative error 1.1e-4, far below bf16 rounding), n added into the exponent field.
// Inputs below -125 (masked scores are -inf) give about 2^-125.
__device__ __forceinline__ uint64_t exp2_poly2(uint64_t a)
{
    float a0, a1;
    unpack_f32x2(a, a0, a1);
    const uint64_t ac = pack_f32x2(fmaxf(a0, -125.0f), fmaxf(a1, -125.0f));
    const uint64_t t = fadd2(ac, pack_f32x2(12582912.0f, 12582912.0f));          // 1.5 * 2^23: integer part lands in the mantissa
    const uint64_t fi = fadd2(t, pack_f32x2(-12582912.0f, -12582912.0f));
    const uint64_t f = ffma2(fi, pack_f32x2(-1.0f, -1.0f), ac);
    uint64_t q = ffma2(pack_f32x2(0.05459282f, 0.05459282f), f, pack_f32x2(0.24221784f, 0.24221784f));
    q = ffma2(q, f, pack_f32x2(0.6933686f, 0.6933686f));
    q = ffma2(q, f, pack_f32x2(1.0f, 1.0f));
    float t0, t1, q0, q1;
    unpack_f32x2(t, t0, t1);
    unpack_f32x2(q, q0, q1);
    const uint32_t r0 = __float_as_uint(q0) + (__float_as_uint(t0) << 23);
    const uint32_t r1 = __float_as_uint(q1) + (__float_as_uint(t1) << 23);
    return pack_f32x2(__uint_as_float(r0), __uint_as_float(r1));
}

// GeLU / GeLU' of two values at once (erf form): the polynomial and scaling steps run as two-wide
// fp32 instructions, the reciprocal and the exponential stay one MUFU op per value.
//   half_tail = erfc(|u|/sqrt2)/2 = (b1 t + ... + b5 t^5) exp(-u^2/2),  t = 1/(1 + p|u|/sqrt2),  b = a/2
__device__ __forceinline__ void normal_cdf_pdf2(float u0, float u1, uint64_t& cdf, uint64_t& e)
{
    const float au0 = fabsf(u0), au1 = fabsf(u1);
    const uint64_t au = pack_f32x2(au0, au1);
    float d0, d1, x0, x1;
    unpack_f32x2(ffma2(au, pack_f32x2(0.23164189f, 0.23164189f), pack_f32x2(1.0f, 1.0f)), d0, d1);      // 1 + p |u| / sqrt2
    unpack_f32x2(fmul2(fmul2(au, au), pack_f32x2(-0.72134752f, -0.72134752f)), x0, x1);                    // -u^2/2 * log2(e)
    const uint64_t t = pack_f32x2(__frcp_rn(d0), __frcp_rn(d1));
    e = pack_f32x2(ex2_approx(x0), ex2_approx(x1));
    uint64_t poly = ffma2(t, pack_f32x2(0.5307027145f, 0.5307027145f), pack_f32x2(-0.7265760135f, -0.7265760135f));
    poly = ffma2(t, poly, pack_f32x2(0.7107068705f, 0.7107068705f));
    poly = ffma2(t, poly, pack_f32x2(-0.142248368f, -0.142248368f));
    poly = ffma2(t, poly, pack_f32x2(0.127414796f, 0.127414796f));
    const uint64_t ht = fmul2(fmul2(poly, t), e);
    // cdf = 1/2 + sign(u) (1/2 - half_tail): the sign of u is OR-ed into 1/2 - half_tail (>= 0), no compare / select
    float g0, g1;
    unpack_f32x2(ffma2(ht, pack_f32x2(-1.0f, -1.0f), pack_f32x2(0.5f, 0.5f)), g0, g1);
    g0 = __uint_as_float(__float_as_uint(g0) | (__float_as_uint(u0) & 0x80000000u));
    g1 = __uint_as_float(__float_as_uint(g1) | (__float_as_uint(u1) & 0x80000000u));
    cdf = fadd2(pack_f32x2(g0, g1), pack_f32x2(0.5f, 0.5f));
}
__device__ __forceinline__ void gelu2_erf(float& u0, float& u1)
{
    uint64_t cdf, e;
    normal_cdf_pdf2(u0, u1, cdf, e);
    unpack_f32x2(fmul2(pack_f32x2(u0, u1), cdf), u0, u1);
}
__device__ __forceinline__ void gelu2(float& u0, float& u1, int act)
{
    if (act == 1) { u0 = gelu_f(u0, 1); u1 = gelu_f(u1, 1); return; }
    gelu2_erf(u0, u1);
}
// g0, g1 *= GeLU'(u0), GeLU'(u1)
__device__ __forceinline__ void gelu_grad_mul2_erf(float& g0, float& g1, float u0, float u1)
{
    uint64_t cdf, e;
    normal_cdf_pdf2(u0, u1, cdf, e);
    const uint64_t up = fmul2(pack_f32x2(u0, u1), pack_f32x2(0.3989422804f, 0.3989422804f));
    unpack_f32x2(fmul2(pack_f32x2(g0, g1), ffma2(up, e, cdf)), g0, g1);
}
__device__ __forceinline__ void gelu_grad_mul2(float& g0, float& g1, float u0, float u1, int act)
{
    if (act == 1) { g0 *= gelu_grad_f(u0, 1); g1 *= gelu_grad_f(u1, 1); return; }
    uint64_t cdf, e;
    normal_cdf_pdf2(u0, u1, cdf, e);
    const uint64_t up = fmul2(pack_f32x2(u0, u1), pack_f32x2(0.3989422804f, 0.3989422804f));
    unpack_f32x2(fmul2(pack_f32x2(g0, g1), ffma2(up, e, cdf)), g0, g1);
}

}  // namespace pw
