// sm_100a batched decode step of the RG-LRU temporal core (bf16 io, head width 256; narrower heads as groups of heads or one
// head per 256 channel slots, see the weight loads below): one new token for each
// of B sequences, recurrent state h [B,D] fp32 and the 3-row conv state [B,3,D] updated in place.
//
// A cluster of two CTAs owns one (head, batch tile) pair.  CTA r of the pair owns channels [128 r, 128 r + 128)
// of the head, both as conv / state channels and as gate output channels:
//   * its 2 x 128 rows of W_a, W_x arrive by tiled TMA in the 128-byte-swizzled K-major layout tcgen05.mma reads
//     (the copy runs while the conv phase works);
//   * all threads do the conv phase for the CTA's own 128 channels: one thread per (sequence, 8 channels) reads
//     x and the three conv-state rows with 16-byte loads, stores the bf16 conv output u as one 16-byte swizzle chunk
//     of the U tile in its own shared memory and writes the shifted conv state back (bit-exact copies) after the
//     hand-over.  Every conv-state element is read and written by exactly one thread.  The CTA's half of the U tile
//     (two K blocks of NB rows x 128 bytes) then goes to the peer CTA as two bulk shared-to-shared copies counted on a
//     barrier of the peer, which only the peer's MMA-issuing thread waits for; a last barrier tells the sender that
//     its copies have been received before it leaves.
//     The rounding remainder u - bf16(u) is kept beside it (own channels only): the gate products take the
//     bf16 value, the term i_t * u_t of Eq. 4 takes bf16(u) + remainder, which is u to 16 mantissa bits;
//   * one thread issues Z^T = W U^T for both gates (M = 128 channels, N = sequences of the tile, K = 256) with
//     fp32 accumulators in tensor memory;
//   * all sixteen warps run the epilogue: channel on the TMEM lane, sequences along the columns; gates, log-space
//     decay and h <- a h + sqrt(1 - a^2) (i u) in fp32, h and y written with lane-contiguous stores.
// Waits on the mbarriers are bounded and end in RGLRU_ERR_TIMEOUT; the only cluster barrier comes before them.
#include <cuda.h>
#include <cuda_bf16.h>

#include "rglru_internal.h"
#include "sm100_ptx.cuh"
#include "sm100_gates.cuh"

namespace rglru {
namespace {

using namespace ptx;

constexpr int DH = 256;        // head width
constexpr int CH = 128;        // channels per CTA
constexpr int NB_MAX = 128;    // sequences per batch tile, at most
constexpr int NTHREADS = 512;
constexpr uint32_t KBLOCK_BYTES = 128 * 128;               // 128 rows x 64 bf16: one K block of an operand tile
constexpr uint32_t SMEM_WA = 0;
constexpr uint32_t SMEM_WX = SMEM_WA + 4 * KBLOCK_BYTES;
constexpr uint32_t SMEM_U = SMEM_WX + 4 * KBLOCK_BYTES;
constexpr uint32_t SMEM_R = SMEM_U + 4 * KBLOCK_BYTES;    // bf16 r_s[NB_MAX][CH]: u - bf16(u) for this CTA's channels
constexpr uint32_t SMEM_BAR = SMEM_R + NB_MAX * CH * 2;   // four mbarriers
constexpr uint32_t SMEM_MISC = SMEM_BAR + 32;             // tmem base
constexpr uint32_t SMEM_TOTAL = SMEM_MISC + 16;
constexpr uint32_t SMEM_ALLOC = SMEM_TOTAL + 1024;
constexpr uint32_t TMEM_COLS = 256;                        // z_a in columns [0, NB), z_x in [128, 128 + NB)

struct DecArgs {
    alignas(64) CUtensorMap tm_wa;   // W_a as [H][256 out][256 in], box 128 out x 64 in, 128-byte swizzle
    alignas(64) CUtensorMap tm_wx;
    FwdArgs f;
    int dh;       // head width of the layer
    int mode;     // 0: a kernel "head" is one layer head in 256 channel slots (width 256, or narrower with the slots beyond the
                  //    width unused); 1 / 2: a group of two 128-wide / four 64-wide heads that fill the 256 channels
    int hstride;  // channels from one kernel "head" to the next (256, or dh in mode 0 with a narrower head)
    int NB;       // sequences per batch tile (multiple of 16)
    int ntile;    // batch tiles
    unsigned long long spin_ns;
};

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(const uint32_t *)&v;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NTHREADS, 1) sm100_decode_kernel(const __grid_constant__ DecArgs p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;   // the same offset in both CTAs of the cluster
    uint8_t *smem = smem_raw + (base - raw_addr);
    // BAR_W: weight bytes; BAR_ACC: accumulators complete; BAR_U: the peer's half of the U tile has landed here;
    // BAR_SENT: the peer has received this CTA's half (nothing of this CTA's shared memory is still being read)
    const uint32_t BAR_W = base + SMEM_BAR, BAR_ACC = BAR_W + 8, BAR_U = BAR_W + 16, BAR_SENT = BAR_W + 24;
    uint32_t *tmem_base_s = (uint32_t *)(smem + SMEM_MISC);

    const FwdArgs &f = p.f;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int B = f.B, D = f.D, NB = p.NB;
    const uint32_t rank = cluster_ctarank();
    const int item = blockIdx.x >> 1, head = item % f.H, tile = item / f.H;
    const int b0 = tile * NB;
    const unsigned long long spin = p.spin_ns;
    int timed_out = 0;
    volatile int no_abort = 0;

    // Programmatic dependent launch: the next kernel on the stream (typically the next decode step) may be scheduled
    // as SMs free up, and runs its own prologue -- barrier set-up, tensor-memory allocation, the weight copies, the
    // conv taps -- while this step is still finishing; it touches x, h and the conv state only after griddepcontrol.wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        mbar_init(BAR_W, 1);
        mbar_init(BAR_ACC, 1);
        mbar_init(BAR_U, 1);
        mbar_init(BAR_SENT, 1);
        mbar_expect_tx(BAR_U, 2u * (uint32_t)NB * 128u);   // two K blocks of NB rows x 128 bytes, sent by the peer
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) { tmem_alloc(smem_u32(tmem_base_s), TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_base_s;
    cluster_arrive();   // the peer must be running before anything is stored into its shared memory

    // ---- this CTA's gate weights: 2 gates x 4 K blocks of [128 out rows x 64 in channels], issued by the last warp so
    //      that the descriptor fetch of the first tiled copy delays nobody's global loads; they are the longest latency
    //      of the step (128 KB per CTA out of L2) and overlap the whole conv phase
    //      Narrower heads (128 or 64 channels) run as groups of 2 or 4 that fill the 256 channels: the group's weight matrix is
    //      block-diagonal, so this CTA's 128 output rows only see K blocks 2 rank and 2 rank + 1 -- the channels it convolves
    //      itself -- and nothing is exchanged with the peer.  With 64-wide heads each of those K blocks holds one head's 64 rows;
    //      the other 64 rows of the block are zeroed by the threads below.
    const int mode = p.mode;
    // first channel of this head in the layer and the number of its 256 channel slots that exist: the slots beyond a narrower
    // head's width get zero weights (the tiled copies read them as out of bounds), zero taps, and are neither loaded nor stored
    const size_t cbase = (size_t)head * p.hstride;
    const int cvalid = mode == 0 ? p.dh : DH;
    if (tid == NTHREADS - 32) {
        if (mode == 0) {
            mbar_expect_tx(BAR_W, 8 * KBLOCK_BYTES);
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
                tma_load_3d(base + SMEM_WA + kb * KBLOCK_BYTES, &p.tm_wa, kb * 64, (int)rank * CH, head, BAR_W);
                tma_load_3d(base + SMEM_WX + kb * KBLOCK_BYTES, &p.tm_wx, kb * 64, (int)rank * CH, head, BAR_W);
            }
        } else if (mode == 1) {
            mbar_expect_tx(BAR_W, 4 * KBLOCK_BYTES);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const uint32_t off = (uint32_t)(2 * (int)rank + j) * KBLOCK_BYTES;
                tma_load_3d(base + SMEM_WA + off, &p.tm_wa, j * 64, 0, 2 * head + (int)rank, BAR_W);
                tma_load_3d(base + SMEM_WX + off, &p.tm_wx, j * 64, 0, 2 * head + (int)rank, BAR_W);
            }
        } else {
            mbar_expect_tx(BAR_W, 2 * KBLOCK_BYTES);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const uint32_t off = (uint32_t)(2 * (int)rank + j) * KBLOCK_BYTES + (uint32_t)j * (KBLOCK_BYTES / 2);
                tma_load_3d(base + SMEM_WA + off, &p.tm_wa, 0, 0, 4 * head + 2 * (int)rank + j, BAR_W);
                tma_load_3d(base + SMEM_WX + off, &p.tm_wx, 0, 0, 4 * head + 2 * (int)rank + j, BAR_W);
            }
        }
    }
    __syncwarp();
    if (mode == 2) {
        // rows of the two K blocks that belong to the other head of this CTA: zero (generic stores; the fence and barrier after
        // the conv phase order them before the MMAs)
        for (int i = tid; i < 4 * (int)(KBLOCK_BYTES / 2 / 16); i += NTHREADS) {
            const int blk = i / (int)(KBLOCK_BYTES / 2 / 16), w16 = i % (int)(KBLOCK_BYTES / 2 / 16);   // blk: gate * 2 + j
            const int j = blk & 1;
            const uint32_t off = (blk >> 1 ? SMEM_WX : SMEM_WA) + (uint32_t)(2 * (int)rank + j) * KBLOCK_BYTES + (uint32_t)(1 - j) * (KBLOCK_BYTES / 2) + (uint32_t)w16 * 16u;
            *(uint4 *)(smem + off) = make_uint4(0u, 0u, 0u, 0u);
        }
    }

    // ---- epilogue constants (parameters only, fetched early): warp (q, kq) owns channels 32 q .. 32 q + 31 and quarter kq
    //      of the tile's sequences
    const int q = warp & 3, kq = warp >> 2;
    const int c_own = q * 32 + lane;
    const int dl = (int)rank * CH + c_own;
    const size_t d = cbase + dl;
    const bool exists = dl < cvalid;   // uniform over the warp (widths are multiples of 32)
    // used after the conv phase: nothing waits on them here
    const float lam = exists ? f.lambda[d] : 0.0f, ba = exists ? f.b_a[d] : 0.0f, bx = exists ? f.b_x[d] : 0.0f;

    // ---- gate products: the K blocks this CTA convolved itself are multiplied while the peer's half is still on its way
    const uint32_t idesc = make_idesc(128, NB);
    auto issue_kblocks = [&](int kb_first, bool first) {   // two K blocks = 8 K steps of 16, both gates
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t koff = (uint32_t)(kb_first + (j >> 2)) * KBLOCK_BYTES + (uint32_t)(j & 3) * 32u;
            const uint64_t bd = make_desc_sw128(base + SMEM_U + koff);
            const uint32_t accum = (first && j == 0) ? 0u : 1u;
            mma_ss(tmem, make_desc_sw128(base + SMEM_WA + koff), bd, idesc, accum);
            mma_ss(tmem + 128, make_desc_sw128(base + SMEM_WX + koff), bd, idesc, accum);
        }
    };
    bool w_ok = true;

    // ---- conv phase: thread = (8-channel chunk c, sequences n = tid/16, tid/16 + 32, ...)
    {
        const int c = tid & 15;
        const int cdl = (int)rank * CH + c * 8;         // channel within the head
        const size_t cd = cbase + cdl;                  // global channel
        const bool cexists = cdl < cvalid;              // the eight channels of this thread exist
        const __nv_bfloat16 *cw = (const __nv_bfloat16 *)f.conv_w;
        uint4 w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j] = cexists ? *(const uint4 *)(cw + (size_t)j * D + cd) : make_uint4(0u, 0u, 0u, 0u);
        float cb[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) cb[e] = f.conv_b && cexists ? f.conv_b[cd + e] : 0.0f;
        const __nv_bfloat16 *x = (const __nv_bfloat16 *)f.x;
        __nv_bfloat16 *cs = (__nv_bfloat16 *)f.cs_out;   // in/out
        const uint32_t u_kb = SMEM_U + (uint32_t)(cdl >> 6) * KBLOCK_BYTES;
        const uint32_t chunk = (uint32_t)(cdl & 63) >> 3;
        // everything above reads only parameters; x and the state may have been written by the kernel just before this
        // one on the stream, whose completion (and visibility of its stores) is awaited here
        asm volatile("griddepcontrol.wait;" ::: "memory");
        // all global loads of the phase are issued before anything waits on them
        constexpr int NIT = NB_MAX / 32;
        uint4 xv[NIT], r0[NIT], r1[NIT], r2[NIT];   // x_t and x_{t-3}, x_{t-2}, x_{t-1} per sequence
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const int n = (tid >> 4) + 32 * i, b = b0 + n;
            if (n < NB && b < B && cexists) {
                xv[i] = *(const uint4 *)(x + (size_t)b * D + cd);
                r0[i] = *(const uint4 *)(cs + ((size_t)b * 3 + 0) * D + cd);
                r1[i] = *(const uint4 *)(cs + ((size_t)b * 3 + 1) * D + cd);
                r2[i] = *(const uint4 *)(cs + ((size_t)b * 3 + 2) * D + cd);
            }
        }
        cluster_wait();   // the peer has set up its barriers
        const uint32_t w0[4] = {w[0].x, w[0].y, w[0].z, w[0].w}, w1[4] = {w[1].x, w[1].y, w[1].z, w[1].w},
                       w2[4] = {w[2].x, w[2].y, w[2].z, w[2].w}, w3[4] = {w[3].x, w[3].y, w[3].z, w[3].w};
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const int n = (tid >> 4) + 32 * i, b = b0 + n;
            if (n >= NB) break;
            uint4 uo = make_uint4(0u, 0u, 0u, 0u);
            if (b < B && cexists) {
                const uint32_t xw[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w}, a0[4] = {r0[i].x, r0[i].y, r0[i].z, r0[i].w},
                               a1[4] = {r1[i].x, r1[i].y, r1[i].z, r1[i].w}, a2[4] = {r2[i].x, r2[i].y, r2[i].z, r2[i].w};
                uint32_t o[4], rem[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float ul = cb[2 * e], uh = cb[2 * e + 1];
                    ul = fmaf(bf_lo(w0[e]), bf_lo(xw[e]), ul); uh = fmaf(bf_hi(w0[e]), bf_hi(xw[e]), uh);
                    ul = fmaf(bf_lo(w1[e]), bf_lo(a2[e]), ul); uh = fmaf(bf_hi(w1[e]), bf_hi(a2[e]), uh);
                    ul = fmaf(bf_lo(w2[e]), bf_lo(a1[e]), ul); uh = fmaf(bf_hi(w2[e]), bf_hi(a1[e]), uh);
                    ul = fmaf(bf_lo(w3[e]), bf_lo(a0[e]), ul); uh = fmaf(bf_hi(w3[e]), bf_hi(a0[e]), uh);
                    o[e] = pack_bf16(ul, uh);
                    rem[e] = pack_bf16(ul - bf_lo(o[e]), uh - bf_hi(o[e]));
                }
                uo = make_uint4(o[0], o[1], o[2], o[3]);
                *(uint4 *)(smem + SMEM_R + (uint32_t)n * (CH * 2) + (uint32_t)c * 16u) = make_uint4(rem[0], rem[1], rem[2], rem[3]);
            }
            *(uint4 *)(smem + u_kb + (uint32_t)n * 128u + ((chunk ^ (uint32_t)(n & 7)) << 4)) = uo;
        }
        fence_async_all();   // generic-proxy writes before the tensor core and the bulk copies read them
        __syncthreads();     // this CTA's half of the U tile is complete in its own shared memory
        // ... and goes to the peer as two bulk copies (one per K block: NB rows of 128 bytes, contiguous), counted on the
        // peer's barrier: nobody but the peer's MMA issuer waits for them
        if (tid == 32 && mode == 0) {
            const uint32_t peer_bar = map_to_cta(BAR_U, rank ^ 1u);
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const uint32_t off = SMEM_U + (uint32_t)((int)rank * 2 + k) * KBLOCK_BYTES;
                bulk_s2peer(map_to_cta(base + off, rank ^ 1u), base + off, (uint32_t)NB * 128u, peer_bar);
            }
        }
        if (tid == 0) {
            w_ok = mbar_wait(BAR_W, 0, spin, &no_abort);
            if (w_ok) {
                tc_fence_after();
                issue_kblocks((int)rank * 2, true);
            } else {
                atomicExch(f.status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT);
            }
        }
        // the conv state moves up by one row: bit-exact copies, stored after the hand-over so that nothing waits on them
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const int n = (tid >> 4) + 32 * i, b = b0 + n;
            if (n < NB && b < B && cexists) {
                *(uint4 *)(cs + ((size_t)b * 3 + 0) * D + cd) = r1[i];
                *(uint4 *)(cs + ((size_t)b * 3 + 1) * D + cd) = r2[i];
                *(uint4 *)(cs + ((size_t)b * 3 + 2) * D + cd) = xv[i];
            }
        }
    }

    const float zl = -lam;
    const float s = f.c * (zl > 0.0f ? zl + log1pf(expf(-zl)) : log1pf(expf(zl)));
    const bool poly = __all_sync(0xffffffffu, s <= S_POLY);
    const f32x2 hba2 = pack2(0.5f * ba, 0.5f * ba), hbx2 = pack2(0.5f * bx, 0.5f * bx), s2 = pack2(s, s);
    const uint8_t *u_col = smem + SMEM_U + (uint32_t)(dl >> 6) * KBLOCK_BYTES + (uint32_t)(dl & 7) * 2u;
    const uint32_t u_chunk = (uint32_t)(dl & 63) >> 3;
    const uint8_t *r_col = smem + SMEM_R + (uint32_t)c_own * 2u;
    float *h = f.h_T;                                 // in/out
    __nv_bfloat16 *y = (__nv_bfloat16 *)f.y;
    const int nq = NB >> 2;                           // multiple of 4
    const uint32_t tm_lane = tmem + ((uint32_t)(q * 32) << 16);
    // the recurrent state of this warp's sequences is fetched while the tensor core works
    float hv[NB_MAX / 4];
#pragma unroll
    for (int j = 0; j < NB_MAX / 4; ++j) {
        const int b = b0 + kq * nq + j;
        hv[j] = (j < nq && b < B && exists) ? h[(size_t)b * D + d] : 0.0f;
    }

    if (tid == 0) {
        // the peer's half of the U tile (waited for even when the weights failed: the peer's copies must have landed
        // before this CTA may leave)
        const bool u_ok = mode != 0 || mbar_wait(BAR_U, 0, spin, &no_abort);
        if (u_ok && mode == 0) mbar_arrive_at(BAR_SENT, rank ^ 1u);
        if (u_ok && w_ok) {
            tc_fence_after();
            if (mode == 0) issue_kblocks((int)(rank ^ 1u) * 2, false);
            tc_commit(BAR_ACC);
        } else if (!u_ok) {
            atomicExch(f.status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT);
        }
    }
    __syncwarp();

    if (!warp_wait(BAR_ACC, 0, spin, &no_abort)) {
        timed_out = 1;
    } else {
        tc_fence_after();
#pragma unroll
        for (int j0 = 0; j0 < NB_MAX / 4; j0 += 4) {
            if (j0 >= nq) break;
            const int n0 = kq * nq + j0;
            float za[4], zx[4];
            tmem_ld4(tm_lane + n0, za);
            tmem_ld4(tm_lane + 128 + n0, zx);
            tmem_ld_wait();
            // two sequences per register pair, two pairs side by side
            f32x2 A2[2], V2[2];
            float u[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int n = n0 + j;
                const uint32_t ub = *(const uint16_t *)(u_col + (uint32_t)n * 128u + ((u_chunk ^ (uint32_t)(n & 7)) << 4));
                const uint32_t rb = *(const uint16_t *)(r_col + (uint32_t)n * (CH * 2));
                u[j] = __uint_as_float(ub << 16) + __uint_as_float(rb << 16);
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) { A2[j] = pack2(za[2 * j], za[2 * j + 1]); V2[j] = pack2(zx[2 * j], zx[2 * j + 1]); }
            if (poly) gate_group<true, 2>(A2, V2, u, hba2, hbx2, s2);
            else gate_group<false, 2>(A2, V2, u, hba2, hbx2, s2);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const f32x2 H2 = fma2(A2[j], pack2(hv[j0 + 2 * j], hv[j0 + 2 * j + 1]), V2[j]);
                const float hn[2] = {lo2(H2), hi2(H2)};
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int b = b0 + n0 + 2 * j + e;
                    if (b < B && exists) {
                        h[(size_t)b * D + d] = hn[e];
                        y[(size_t)b * D + d] = __float2bfloat16_rn(hn[e]);
                    }
                }
            }
        }
    }
    if (__any_sync(0xffffffffu, timed_out) && lane == 0) atomicExch(f.status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT);
    if (timed_out) {   // let the weight copies and MMAs in flight land before shared and tensor memory are given back
        const uint64_t tw = gtimer();
        while (gtimer() - tw < 50000ull) __nanosleep(1000);
    }

    // the peer has received this CTA's half of the U tile: its bulk copies no longer read this shared memory
    if (tid == 0 && !timed_out && mode == 0) mbar_wait(BAR_SENT, 0, spin, &no_abort);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

int num_sms() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) return n;
    return 148;
}

}  // namespace

// Head width 256, or 128 / 64 with the heads filling whole 256-channel groups.
// Any other multiple of 32 below 256: one head per 256 channel slots.
namespace {
inline bool grouped_heads(int D, int H) { const int dh = D / H; return dh == DH || ((dh == 128 || dh == 64) && D % DH == 0); }
}  // namespace
bool sm100_decode_supported(int B, int D, int H, int io) {
    if (io != RGLRU_BF16 || B <= 0 || H <= 0 || D % H != 0) return false;
    const int dh = D / H;
    return grouped_heads(D, H) || (dh < DH && dh % 32 == 0);
}

cudaError_t sm100_decode(const FwdArgs &a, cudaStream_t st) {
    static PerDeviceOptIn opt_in;
    cudaError_t e = opt_in.ensure(sm100_decode_kernel, (int)SMEM_ALLOC);
    if (e != cudaSuccess) return e;
    DecArgs p;
    const int dh = a.D / a.H;
    const bool grouped = grouped_heads(a.D, a.H);
    const int G = grouped ? a.D / DH : a.H;   // 256-channel groups of heads, or heads of another width: the kernel's unit
    const int mode = !grouped || dh == DH ? 0 : (dh == 128 ? 1 : 2);
    const uint32_t box_rows = mode == 2 ? 64u : (uint32_t)CH;
    if (!encode_bf16_map_3d(&p.tm_wa, a.W_a, (uint64_t)dh, (uint64_t)dh, (uint64_t)a.H, 64, box_rows, true) ||
        !encode_bf16_map_3d(&p.tm_wx, a.W_x, (uint64_t)dh, (uint64_t)dh, (uint64_t)a.H, 64, box_rows, true))
        return cudaErrorNotSupported;
    p.f = a;
    p.f.H = G;
    p.dh = dh;
    p.mode = mode;
    p.hstride = grouped ? DH : dh;
    // batch tile: as few tiles per head as fill the SM pairs once, rounded to the MMA's N granularity
    const int pairs = num_sms() / 2;
    const int tiles_wanted = pairs / G > 0 ? pairs / G : 1;
    int NB = (a.B + tiles_wanted - 1) / tiles_wanted;
    NB = ((NB + 15) / 16) * 16;
    if (NB > NB_MAX) NB = NB_MAX;
    if (NB < 16) NB = 16;
    p.NB = NB;
    p.ntile = (a.B + NB - 1) / NB;
    p.spin_ns = g_spin_limit_ns;
    dim3 grid(2u * (unsigned)G * (unsigned)p.ntile), block(NTHREADS);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = SMEM_ALLOC; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, sm100_decode_kernel, p);
}

}  // namespace rglru
