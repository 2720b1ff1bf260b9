// PTX wrappers for the sm_100a kernels: mbarriers, bulk / tiled TMA copies, tensor memory, tcgen05.mma,
// packed fp32x2 arithmetic and the approximate transcendental instructions.  Device code only.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rglru {
namespace ptx {

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// Nanosecond timer shared by all SMs.  The 64-bit value is assembled from two 32-bit halves that are re-read until
// the high half is stable, so a reading taken while the low half wraps (every 4.29 s) cannot be off by 2^32 ns.
__device__ __forceinline__ uint64_t gtimer() {
    uint32_t hi0, lo, hi1;
    do {
        asm volatile("mov.u32 %0, %%globaltimer_hi;" : "=r"(hi0));
        asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(lo));
        asm volatile("mov.u32 %0, %%globaltimer_hi;" : "=r"(hi1));
    } while (hi0 != hi1);
    return ((uint64_t)hi1 << 32) | lo;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One test of the barrier phase.  The thread may be suspended until the phase completes or the hinted time has passed,
// whichever comes first.
constexpr uint32_t MBAR_SUSPEND_NS = 20000;
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.b32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "n"(MBAR_SUSPEND_NS) : "memory");
    return ok != 0;
}
// Up to 256 tests in a loop of three instructions (a suspended thread is woken by unrelated barrier traffic as well, so
// tests are frequent and the loop around them must be cheap).
__device__ __forceinline__ bool mbar_try256(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\n.reg .b32 n;\nmov.b32 n, 256;\nMBT_LOOP:\n"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n@p bra MBT_DONE;\n"
                 "sub.u32 n, n, 1;\nsetp.ne.u32 p, n, 0;\n@p bra MBT_LOOP;\nsetp.ne.u32 p, n, 0;\n"
                 "MBT_DONE:\nselp.b32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "n"(MBAR_SUSPEND_NS) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or the CTA is aborting; the abort flag and the global timer are
// consulted once every 256 tests.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    if (mbar_try256(bar, parity)) return true;
    const uint64_t t0 = gtimer();
    for (;;) {
        if (mbar_try256(bar, parity)) return true;
        if (*abort_flag || gtimer() - t0 > limit_ns) return false;
    }
}
// Bounded wait that never suspends the thread: for hand-offs that are normally tens of cycles away, where the wake-up time of a
// suspended thread would dominate.
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    uint32_t ok;
    uint64_t t0 = 0;
    for (uint32_t n = 0;; ++n) {
        asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.b32 %0, 1, 0, p;\n}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((n & 1023u) == 1023u) {
            if (*abort_flag) return false;
            const uint64_t t = gtimer();
            if (t0 == 0) t0 = t;
            else if (t - t0 > limit_ns) return false;
        }
    }
}
__device__ __forceinline__ bool warp_wait_spin(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    return __all_sync(0xffffffffu, mbar_wait_spin(bar, parity, limit_ns, abort_flag));
}
// Bounded wait for something that is normally many microseconds away (a ring slot several stages ahead): the thread sleeps
// between tests instead of being woken by every barrier event of the CTA.
__device__ __forceinline__ bool mbar_wait_far(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    uint32_t ok;
    uint64_t t0 = 0;
    for (uint32_t n = 0;; ++n) {
        asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.b32 %0, 1, 0, p;\n}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        __nanosleep(2000);
        if ((n & 15u) == 15u) {
            if (*abort_flag) return false;
            const uint64_t t = gtimer();
            if (t0 == 0) t0 = t;
            else if (t - t0 > limit_ns) return false;
        }
    }
}
__device__ __forceinline__ bool warp_wait_far(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    return __all_sync(0xffffffffu, mbar_wait_far(bar, parity, limit_ns, abort_flag));
}
// All lanes wait (a wait or sleep executed by part of a warp returns at once, as measured); the verdict is made
// warp-uniform so that a warp never splits on a timeout.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, limit_ns, abort_flag));
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]^T, kind::f16 (A and B of one 16-bit type chosen by the instruction descriptor,
// fp32 accumulate), one CTA
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
// Two fp32 values in an aligned register pair; arithmetic through the packed-fp32 builtins (fma.rn.f32x2 and friends).
typedef float2 f32x2;
// D[tmem] (+)= A[smem] * B[smem]^T, kind::f16 (A and B of one 16-bit type, fp32 accumulate), one CTA
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
// 8 consecutive columns of this thread's lane
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float *v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr) : "memory");
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[j]);
}
// 4 consecutive columns of this thread's lane
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, float *v) {
    uint32_t r[4];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = __uint_as_float(r[j]);
}
// ---- thread-block clusters and distributed shared memory
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t cta_rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta_rank)); return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, uint4 v) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
// 32 consecutive columns of this thread's lane as 16 register pairs (column 2j in the low half)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, f32x2 *v) {
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
                   "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
                   "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]),
                   "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st8(uint32_t taddr, uint4 lo, uint4 hi) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// shared -> global bulk copy, tracked by this thread's bulk async-group
__device__ __forceinline__ void bulk_s2g(void *dst, uint32_t src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}
// one tiled TMA load of a [rows x channels] box at (channel c0, token t, sequence b); rows outside [0, T) read as zero
__device__ __forceinline__ void tma_load_3d(uint32_t dst_smem, const CUtensorMap *tm, int c0, int t, int b, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst_smem), "l"(tm), "r"(c0), "r"(t), "r"(b), "r"(bar) : "memory");
}
// one tiled TMA store; rows at or beyond T are clipped by the tensor bounds
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *tm, int c0, int t, int b, uint32_t src_smem) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(tm), "r"(c0), "r"(t), "r"(b), "r"(src_smem) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// K-major, 128B-swizzled shared-memory operand: rows of 128 B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}
// MN-major, 128B-swizzled shared-memory operand: rows (one K index each) of 64 elements of the M or N dimension = 128 B,
// 8-row groups 1024 B apart along K (stride offset), 64-element blocks of the M / N dimension `block_bytes` apart (leading
// offset).  This is what a tiled copy with the M / N dimension innermost and a 128-byte swizzle leaves in shared memory.
__device__ __forceinline__ uint64_t make_desc_sw128_mn(uint32_t saddr, uint32_t block_bytes) {
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)((block_bytes >> 4) & 0x3FFF) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// kind::f16 instruction descriptor: fp32 accumulator, fp16 A and B, both MN-major (bits 15 and 16), M x N
__host__ __device__ constexpr uint32_t make_idesc_f16_mn(int M, int N) {
    return (1u << 4) | (1u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// kind::f16 instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, M x N
__host__ __device__ constexpr uint32_t make_idesc_f16(int M, int N) {
    return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// two fp32 -> packed fp16 (lo in the low half), round to nearest even, finite overflow saturates to +-65504
__device__ __forceinline__ uint32_t pack_f16_sat(float lo, float hi) {
    uint32_t r; asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo)); return r;
}
__device__ __forceinline__ float f16_bits_to_f32(uint16_t h) { float r; asm("cvt.f32.f16 %0, %1;" : "=f"(r) : "h"(h)); return r; }
// The same, kept in program order with respect to the other volatile statements around it: a conversion placed before a
// barrier arrive proves that the load which produced its operand has completed by then.
__device__ __forceinline__ float f16_bits_to_f32_ordered(uint16_t h) { float r; asm volatile("cvt.f32.f16 %0, %1;" : "=f"(r) : "h"(h)); return r; }
// the same descriptor with bf16 A and B
__host__ __device__ constexpr uint32_t make_idesc(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---- packed fp32x2 arithmetic (one issue slot for two lanes' worth of FP32 work)
__device__ __forceinline__ f32x2 pack2(float lo, float hi) { return make_float2(lo, hi); }
__device__ __forceinline__ float lo2(f32x2 v) { return v.x; }
__device__ __forceinline__ float hi2(f32x2 v) { return v.y; }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float tanh_approx(float x) { float y; asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float sqrt_approx(float x) { float y; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float ex2_approx(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }


// ---- CTA pairs (cluster of two): tensor memory, MMA and barriers of the two-CTA form of tcgen05
// Both CTAs of the pair execute the allocation, the relinquish and the deallocation, each with one warp of the same index.
__device__ __forceinline__ void tmem_alloc2(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]^T over the pair: M = 256 (rows 0..127 in the leader's tensor memory, 128..255 in the
// peer's), N tokens of which each CTA's shared memory holds half.  Issued by one thread of the leader CTA.
__device__ __forceinline__ void mma_ts2(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
// Completion of this thread's earlier pair MMAs arrives once on the barrier at the same offset in every CTA of the mask.
__device__ __forceinline__ void tc_commit2(uint32_t bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(cta_mask) : "memory");
}
// Arrive on the barrier at this shared-memory offset in CTA `cta` of the cluster (this CTA included).  The default
// semantics (release at CTA scope) are used on purpose: a release at cluster scope was measured at 1.5-2 k cycles per
// arrive.  What the arrivals publish is ordered by other means: tensor-memory accesses by tcgen05.fence, shared-memory
// tiles for the tensor core by fence.proxy.async, and "done reading" signals publish nothing.
__device__ __forceinline__ void mbar_arrive_at(uint32_t bar, uint32_t cta) {
    asm volatile("{\n.reg .b32 ra;\nmapa.shared::cluster.u32 ra, %0, %1;\nmbarrier.arrive.shared::cluster.b64 _, [ra];\n}"
                 ::"r"(bar), "r"(cta) : "memory");
}
__device__ __forceinline__ bool mbar_try_cl(uint32_t bar, uint32_t parity) { return mbar_try(bar, parity); }
// Bounded wait on a barrier that threads of the peer CTA arrive on (same code as mbar_wait: see mbar_arrive_at).
__device__ __forceinline__ bool mbar_wait_cl(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    return mbar_wait(bar, parity, limit_ns, abort_flag);
}
__device__ __forceinline__ bool warp_wait_cl(uint32_t bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag) {
    return warp_wait(bar, parity, limit_ns, abort_flag);
}
// bulk copy from this CTA's shared memory into a peer's (addresses of the peer in the cluster window); the bytes are counted
// on a barrier of the peer
__device__ __forceinline__ void bulk_s2peer(uint32_t dst_cluster, uint32_t src_smem, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(src_smem), "r"(bytes), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ uint32_t ld_cluster_u16(uint32_t cluster_addr) {
    uint16_t v; asm volatile("ld.shared::cluster.u16 %0, [%1];" : "=h"(v) : "r"(cluster_addr) : "memory"); return v;
}
__device__ __forceinline__ uint32_t ld_shared_u16(uint32_t addr) {
    uint16_t v; asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr) : "memory"); return v;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// 16 consecutive columns of this thread's lane as 8 register pairs (column 2j in the low half)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, f32x2 *v) {
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
                   "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const f32x2 *v) {
    uint32_t r[16];
#pragma unroll
    for (int j = 0; j < 8; ++j) { r[2 * j] = __float_as_uint(v[j].x); r[2 * j + 1] = __float_as_uint(v[j].y); }
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
                   "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
// 16 consecutive columns as plain floats
__device__ __forceinline__ void tmem_ld16f(uint32_t taddr, float *v) {
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
                   "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
}
// 32 consecutive columns from 16 register pairs
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const f32x2 *v) {
    uint32_t r[32];
#pragma unroll
    for (int j = 0; j < 16; ++j) { r[2 * j] = __float_as_uint(v[j].x); r[2 * j + 1] = __float_as_uint(v[j].y); }
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
                   "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
                   "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
                   "r"(r[30]), "r"(r[31]) : "memory");
}
// 8 consecutive columns of this thread's lane as 4 register pairs (column 2j in the low half), and the matching store
__device__ __forceinline__ void tmem_ld8p(uint32_t taddr, f32x2 *v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr) : "memory");
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
}
__device__ __forceinline__ void tmem_st8p(uint32_t taddr, const f32x2 *v) {
    uint32_t r[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) { r[2 * j] = __float_as_uint(v[j].x); r[2 * j + 1] = __float_as_uint(v[j].y); }
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }

}  // namespace ptx
}  // namespace rglru
