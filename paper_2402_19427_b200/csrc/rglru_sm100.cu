// sm_100a fused prefill for the RG-LRU temporal core (bf16 io, head width 256; narrower heads, any multiple of 32, run as
// groups of 256 / width consecutive heads in the 256 channel slots, with a block-diagonal weight matrix).
//
// A head is owned by a pair of CTAs (a cluster of two, one CTA per SM).  CTA r of the pair keeps rows
// [128 r, 128 r + 128) of W_a and W_x resident in its tensor memory as the A operand of the two-CTA form of
// tcgen05.mma (M = 256 over the pair) for the whole launch.  The pair walks tiles of 64 tokens; CTA r convolves tokens
// [32 r, 32 r + 32) of a tile for all 256 channels of the head, so the Conv1D runs once per element:
//   loader warp    35 token rows (32 + 3 of history) of the head's x -> shared memory, one tiled TMA copy per tile
//   conv warps     causal width-4 depthwise conv in fp32 -> fp16 tile U[32 tokens][256 ch] in the K-major
//                  128B-swizzled layout tcgen05.mma reads as this CTA's half of the B operand
//   MMA warps      (leader CTA only) Z_a^T = W_a U^T and Z_x^T = W_x U^T, N = 64 tokens, K = 256: channels on TMEM
//                  lanes, time along TMEM columns, two accumulator buffers used alternately
//   gate warps     tcgen05.ld half a tile of (z_a, z_x), u from the U tile of the CTA that convolved the token (its own
//                  or the peer's through distributed shared memory), gates, log-space decay, input scale, then the
//                  recurrence over the 32 tokens from zero state; (prod a, h from zero) written back over (z_a, z_x)
//                  with tcgen05.st.  They carry no state between tiles and never wait for one.
//   scan warps     hold the exact state: y_t = (h_t from zero) + (prod a up to t) h_in in fp32 for each half tile,
//                  y through a per-warp tiled store, h_in of the next tile from the half tiles' end values
// x is read from HBM once, y written once; u, r, i, a never leave the pair.
//
// Time is split across pairs so that every SM has work even for a single long sequence: sequences that cannot be
// dealt out whole go to the S pairs of a head tile by tile, round-robin.  The scan warp folds such a tile to the
// aggregate (prod a_t, h_end from zero state), publishes it, and obtains its incoming state from its own previous
// tile plus the S-1 aggregates published by the other pairs (decoupled look-back); only then does it run the scan.
// Waits are bounded and end in RGLRU_ERR_TIMEOUT; the launch is cooperative so that all CTAs are co-resident.
#include <cooperative_groups.h>
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <chrono>
#include <mutex>
#include <type_traits>

#include "rglru_internal.h"
#include "sm100_ptx.cuh"
#include "sm100_gates.cuh"

namespace rglru {
namespace {

constexpr int DH = 256;            // head width handled by this kernel
constexpr int CH = 128;            // channels per CTA (half a head)
constexpr int TILE = 64;           // tokens per MMA tile of a pair
constexpr int HALF = 32;           // tokens of a tile one CTA convolves (one TMA slab)
constexpr int SLAB_ROWS = HALF + 3;
constexpr int XS = 4;              // x slab ring depth
constexpr int US = 6;              // U tile stages
constexpr int NUM_THREADS = 640;
constexpr int MAX_S = 16;          // at most this many pairs share one head's time axis
constexpr int LOOKBACK_BATCH = 8;  // carry records requested at once by the look-back
constexpr uint32_t U_STAGE_BYTES = HALF * DH * 2;          // 16384
constexpr uint32_t U_KBLOCK_BYTES = HALF * 128;            // 4096: one 64-channel K block
constexpr uint32_t X_ROW_BYTES = DH * 2;                   // 512
constexpr uint32_t X_SLAB_BYTES = SLAB_ROWS * X_ROW_BYTES; // 17920
constexpr uint32_t SMEM_U = 0;
constexpr uint32_t SMEM_X = SMEM_U + US * U_STAGE_BYTES;
constexpr uint32_t Y_BUF_BYTES = TILE * 32 * 2;            // 4096: one scan warp's 64 tokens x 32 channels
constexpr uint32_t SMEM_Y = SMEM_X + XS * X_SLAB_BYTES;    // bf16 y_s[4 warps][2 buffers][64][32], staged for tiled stores
constexpr uint32_t SMEM_AGG = SMEM_Y + 4 * 2 * Y_BUF_BYTES;   // float2 agg_s[2 buffers][2 half tiles][128 channels]
constexpr uint32_t SMEM_BAR = SMEM_AGG + 2 * 2 * CH * 8;
constexpr int NUM_BARS = 2 * XS + 2 * US + 4 + 8 + 1 + 4;
constexpr uint32_t SMEM_MISC = SMEM_BAR + NUM_BARS * 8;    // tmem base, abort flag
constexpr uint32_t SMEM_TOTAL = SMEM_MISC + 16;
constexpr uint32_t SMEM_ALLOC = SMEM_TOTAL + 1024;         // slack for 1024-byte alignment

// TMEM columns: accumulator buffer bf holds z_a (later a_t) in [128 bf, 128 bf + 64) and z_x (later v_t) in the next 64
constexpr uint32_t TM_W_A = 256, TM_W_X = 384;
__host__ __device__ constexpr uint32_t tm_acc(int bf, int gate) { return (uint32_t)(bf * 128 + gate * 64); }

// y * GeLU(g) for two tokens at once, GeLU(v) = v Phi(v) = v (1 + erf(v / sqrt 2)) / 2 (Section 2.3).  erf by the rational
// approximation 7.1.26 of Abramowitz & Stegun (|error| < 1.5e-7):
// 1 - erf(z) = t (a1 + t (a2 + t (a3 + t (a4 + t a5)))) exp(-z^2), t = 1 / (1 + p z), z >= 0.
__device__ __forceinline__ f32x2 gelu_times2(f32x2 y, float g0, float g1) {
    const f32x2 g = pack2(g0, g1);
    const f32x2 z = mul2(pack2(fabsf(g0), fabsf(g1)), pack2(0.70710678f, 0.70710678f));
    const f32x2 den = fma2(z, pack2(0.3275911f, 0.3275911f), pack2(1.0f, 1.0f));
    const f32x2 t = pack2(__fdividef(1.0f, lo2(den)), __fdividef(1.0f, hi2(den)));
    f32x2 q = fma2(t, pack2(1.061405429f, 1.061405429f), pack2(-1.453152027f, -1.453152027f));
    q = fma2(q, t, pack2(1.421413741f, 1.421413741f));
    q = fma2(q, t, pack2(-0.284496736f, -0.284496736f));
    q = fma2(q, t, pack2(0.254829592f, 0.254829592f));
    const f32x2 ez = mul2(mul2(z, z), pack2(-1.44269504f, -1.44269504f));
    q = mul2(mul2(q, t), pack2(ex2_approx(lo2(ez)), ex2_approx(hi2(ez))));   // 1 - erf(z)
    const f32x2 two_phi = pack2(g0 >= 0.0f ? 2.0f - lo2(q) : lo2(q), g1 >= 0.0f ? 2.0f - hi2(q) : hi2(q));   // 1 + erf(g / sqrt 2)
    return mul2(y, mul2(mul2(g, pack2(0.5f, 0.5f)), two_phi));
}

struct Sm100Args {
    // x as [B][T][D] with a box of SLAB_ROWS token rows x one head; y with a box of TILE rows x 32 channels
    alignas(64) CUtensorMap tm_x;
    alignas(64) CUtensorMap tm_y;
    alignas(64) CUtensorMap tm_g;   // gate branch, same geometry as y (encoded only when the call has one)
    FwdArgs f;
    int dh;            // width of a head of the layer, a multiple of 32 up to 256.  A "head" below is a group of k = 256 / dh
                       // (rounded down) consecutive layer heads: its weight matrices are block-diagonal with k blocks
    int hstride;       // channels from one "head" of the kernel to the next: k dh
    int cvalid;        // channel slots of a "head" that exist: k dh (fewer in the layer's last group when k does not divide H)
    int S;             // pairs per head (time split factor)
    int tps;           // tiles per sequence
    int tiles_total;   // B * tps
    uint32_t tag;      // validity tag of this call's aggregate records
    uint32_t tag_wait; // the tag the look-back waits for: `tag`, or a value nobody publishes under the failure-path test flag
    uint4 *agg;        // [H*2][tiles_total][128] records {P, tag, h_loc, tag}
    unsigned long long spin_ns;
};

using namespace ptx;

// MERGED: the call has a gate branch and writes y_t = h_t GeLU(branch_t); a separate instantiation so that the plain forward
// carries none of its code.
template <bool MERGED>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1) sm100_prefill_kernel(const __grid_constant__ Sm100Args p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    const uint32_t bar0 = base + SMEM_BAR;
    // barrier indices
    auto BAR_XFULL = [&](int s) { return bar0 + 8u * s; };
    auto BAR_XEMPTY = [&](int s) { return bar0 + 8u * (XS + s); };
    auto BAR_UFULL = [&](int s) { return bar0 + 8u * (2 * XS + s); };              // used in the leader CTA only
    auto BAR_UEMPTY = [&](int s) { return bar0 + 8u * (2 * XS + US + s); };
    auto BAR_ACCFULL = [&](int bf) { return bar0 + 8u * (2 * XS + 2 * US + bf); };
    auto BAR_ACCEMPTY = [&](int bf) { return bar0 + 8u * (2 * XS + 2 * US + 2 + bf); };   // leader CTA only
    auto BAR_GDONE = [&](int bf, int q) { return bar0 + 8u * (2 * XS + 2 * US + 4 + bf * 4 + q); };
    const uint32_t BAR_WREADY = bar0 + 8u * (2 * XS + 2 * US + 12);               // leader CTA only: both CTAs' weights are in tensor memory
    auto BAR_BRANCH = [&](int q) { return bar0 + 8u * (2 * XS + 2 * US + 13 + q); };   // scan warp q's block of the gate branch has landed
    uint32_t *tmem_base_s = (uint32_t *)(smem + SMEM_MISC);
    volatile int *abort_flag = (volatile int *)(smem + SMEM_MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const FwdArgs &f = p.f;
    const int T = f.T, D = f.D, S = p.S;
    // CTA `rank` of the pair owns output channels [128 rank, 128 rank + 128) of the head and convolves tokens
    // [32 rank, 32 rank + 32) of every tile for both CTAs.  Rank 0 is the leader: it issues the MMAs of the pair.
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int head = pair / S, kcta = pair % S;
    const int group = head * 2 + (int)rank;   // index of this half-head's carry records
    // First channel of this head (a group of k = 256 / width layer heads) in the layer, and how many of its 256 channel slots
    // exist.  The slots beyond k width read whatever follows in memory (the next group's channels, or zeros past the end of
    // the tensor), their weights are zero in both directions, and nothing of them is written.
    const int cbase = head * p.hstride, cvalid = min(p.cvalid, D - cbase);   // the layer's last group may hold fewer heads
    const uint32_t peer_abort = map_to_cta(base + SMEM_MISC + 4, rank ^ 1u);
    auto record_timeout = [&]() {
        *abort_flag = 1;
        st_cluster_u32(peer_abort, 1u);   // the peer would otherwise run into its own limit waiting for this CTA
        atomicExch(f.status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT);
    };
    // Work of this pair.  Sequences are dealt out whole where that keeps the S pairs of the head balanced: pair kcta
    // gets sequences kcta, kcta + S, ... of the first (B / S) * S ones and walks each from start to end, so a tile's
    // incoming state is simply the state the pair itself reached ("local" tiles: no record, no look-back).  The B % S
    // sequences left over are split in time, tile g of them going to pair g % S ("shared" tiles, decoupled look-back).
    // Shared tiles come first, so that the S pairs pass through them in step.
    const int B_whole = (f.B / S) * S, shared_tiles = (f.B - B_whole) * p.tps;
    const int n_shared = kcta < shared_tiles ? (shared_tiles - kcta + S - 1) / S : 0;
    const int n_my_tiles = n_shared + (B_whole / S) * p.tps;
    // The pair's tiles in order: tile_first gives (sequence b, tile ti within it) of tile 0, tile_next steps from tile
    // `it` to tile `it + 1`; tile `it` is a shared one when it < n_shared.  Tile `it` uses U stage it % US and
    // accumulator buffer it & 1 in both CTAs.
    auto tile_first = [&](int &b, int &ti) {
        if (n_shared > 0) { b = B_whole + kcta / p.tps; ti = kcta % p.tps; } else { b = kcta; ti = 0; }
    };
    auto tile_next = [&](int it, int &b, int &ti) {
        if (it + 1 < n_shared) {
            ti += S;
            while (ti >= p.tps) { ti -= p.tps; ++b; }
        } else if (it + 1 == n_shared) {
            b = kcta; ti = 0;
        } else if (++ti == p.tps) {
            ti = 0; b += S;
        }
    };
    const unsigned long long spin = p.spin_ns;

    if (tid == 0) {
        for (int s = 0; s < XS; ++s) { mbar_init(BAR_XFULL(s), 1); mbar_init(BAR_XEMPTY(s), 4); }
        // U stage full: the four conv warps of both CTAs (counted in the leader).  Free again: both MMA issuers' commits plus
        // the four gate warps of each CTA that read u from this CTA's stage.
        for (int s = 0; s < US; ++s) { mbar_init(BAR_UFULL(s), 8); mbar_init(BAR_UEMPTY(s), 10); }
        for (int bf = 0; bf < 2; ++bf) {
            mbar_init(BAR_ACCFULL(bf), 2);    // one commit per MMA issuer
            mbar_init(BAR_ACCEMPTY(bf), 8);   // the four scan warps of both CTAs
            for (int q = 0; q < 4; ++q) mbar_init(BAR_GDONE(bf, q), 2);
        }
        mbar_init(BAR_WREADY, 16);
        for (int q = 0; q < 4; ++q) mbar_init(BAR_BRANCH(q), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) { tmem_alloc2(smem_u32(tmem_base_s), 512); tmem_relinquish2(); }
    tc_fence_before();
    cluster_arrive();   // the peer's barriers must exist before anything arrives on them
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem = *tmem_base_s;

    // Gate weights of this half-head into tensor memory: lane = output channel, 32-bit column j holds
    // input channels 2j (low half) and 2j+1 (high half).  The tensor core multiplies them with the conv output
    // u, which is kept in fp16 (11 significant bits instead of bf16's 8, because u also enters i_t * u_t of
    // Eq. 4 directly), and both operands of one MMA must have one type: the bf16 weights are converted to
    // fp16 here, which is exact for every weight of magnitude within [2^-14, 65504] and rounds tinier ones
    // to a multiple of 2^-24.
    if (warp >= 8 && warp < 16) {
        const int q = warp & 3, g = (warp - 8) >> 2;  // g = 0: W_a, 1: W_x
        const __nv_bfloat16 *W = (const __nv_bfloat16 *)(g ? f.W_x : f.W_a);
        // Narrower heads (128 or 64 channels) run as groups of 2 or 4 heads that fill the 256 x 256 block: the block is then
        // block-diagonal, and a row holds its own head's weights in that head's input channels and zeros elsewhere.
        const int dh = p.dh, row_in_group = (int)rank * CH + q * 32 + lane;
        const int sub = row_in_group / dh;                     // head of the group this output channel belongs to
        const uint4 *row = (const uint4 *)(W + ((size_t)cbase + row_in_group) * dh);   // (head * 256 / dh + sub) * dh + row_in_group % dh rows of dh
        // the 16-byte chunks of the 256 input channels that are this head's (none for a channel slot that does not exist)
        const int c_first = sub * (dh >> 3), c_count = row_in_group < cvalid ? dh >> 3 : 0;
        const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (g ? TM_W_X : TM_W_A);
        auto cvt2 = [](uint32_t w) { return pack_f16_sat(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u)); };
        const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 4
        for (int c = 0; c < 16; ++c) {
            const int c0 = 2 * c - c_first, c1 = c0 + 1;
            uint4 lo = (c0 >= 0 && c0 < c_count) ? __ldg(row + c0) : zero4, hi = (c1 >= 0 && c1 < c_count) ? __ldg(row + c1) : zero4;
            lo.x = cvt2(lo.x); lo.y = cvt2(lo.y); lo.z = cvt2(lo.z); lo.w = cvt2(lo.w);
            hi.x = cvt2(hi.x); hi.y = cvt2(hi.y); hi.z = cvt2(hi.z); hi.w = cvt2(hi.w);
            tmem_st8(taddr + c * 8, lo, hi);
        }
        tmem_st_wait();
        // only the MMA issuers wait for the weights: loads and the conv of the first tiles run meanwhile
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_at(BAR_WREADY, 0);
    }

    // Register budget per warpgroup (the four warps of a group execute the same setmaxnreg; the increases draw on
    // what the decreases release: 128 (96-64) + 128 (96-40) = 256 (112-96) + 128 (152-96)):
    // conv producers 64, loader / MMA issuers / idle 40, gate warps 112, scan warps 152.
    if (warp < 4) {
        // ================================================================ conv producers
        reg_dec<64>();
        const int pblk = warp;                       // K block = 64 channels of the head
        const int l16 = lane & 15, tg = lane >> 4;   // 4-channel chunk, token group of 16
        const int hc = pblk * 64 + l16 * 4;          // channel within the head
        const __nv_bfloat16 *cw = (const __nv_bfloat16 *)f.conv_w;
        f32x2 w01[4], w23[4], b01, b23;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const __nv_bfloat16 *wp = cw + (size_t)j * D + cbase + hc;
            if (hc < cvalid) {
                w01[j] = pack2(__bfloat162float(wp[0]), __bfloat162float(wp[1]));
                w23[j] = pack2(__bfloat162float(wp[2]), __bfloat162float(wp[3]));
            } else { w01[j] = pack2(0.f, 0.f); w23[j] = w01[j]; }
        }
        if (f.conv_b && hc < cvalid) {
            const float *bp = f.conv_b + cbase + hc;
            b01 = pack2(bp[0], bp[1]); b23 = pack2(bp[2], bp[3]);
        } else { b01 = pack2(0.f, 0.f); b23 = b01; }
        // this thread's 16 tokens are rows 16 tg .. 16 tg + 15 of the slab (plus three rows of history) and of the U tile;
        // U row r keeps its 16-byte chunk c at position c ^ (r & 7) (128-byte swizzle)
        const uint32_t x_thread_off = (uint32_t)hc * 2 + (uint32_t)(tg * 16) * X_ROW_BYTES;
        const uint32_t u_chunk = (uint32_t)(l16 >> 1);
        const uint32_t u_thread_off = SMEM_U + pblk * U_KBLOCK_BYTES + (uint32_t)(l16 & 1) * 8 + (uint32_t)(tg * 16) * 128u;
        uint32_t sw[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) sw[m] = u_thread_off + ((u_chunk ^ (uint32_t)m) << 4);
        bool ok = true;
        for (int it = 0; it < n_my_tiles; ++it) {
            const int st = it % US, slot = it % XS;
            ok = warp_wait_far(BAR_UEMPTY(st), ((it / US) & 1) ^ 1, spin, abort_flag);
            if (!ok) break;
            ok = warp_wait(BAR_XFULL(slot), (it / XS) & 1, spin, abort_flag);
            if (!ok) break;
            const uint8_t *xs = smem + SMEM_X + slot * X_SLAB_BYTES + x_thread_off;
            uint8_t *us = smem + st * U_STAGE_BYTES;
            auto load_row = [&](const uint8_t *row, f32x2 &v01, f32x2 &v23) {
                const uint2 w = *(const uint2 *)row;
                v01 = pack2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u));
                v23 = pack2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
            };
            // Rows before the sequence start and at or beyond its end were filled with zeros by the copy, so all 16 tokens
            // are convolved unconditionally; tokens that do not exist produce rows nobody uses.
            // Four tokens at a time, tap by tap, so that eight independent FMA chains are in flight.  The loop over the
            // halves of the 16 tokens stays rolled: the kernel's roles together must fit the instruction cache.
            f32x2 h01[3], h23[3];   // x_{t-3}, x_{t-2}, x_{t-1}
#pragma unroll
            for (int k = 0; k < 3; ++k) load_row(xs + k * X_ROW_BYTES, h01[k], h23[k]);
#pragma unroll 1
            for (int trip = 0; trip < 2; ++trip) {
                const uint8_t *xr = xs + (uint32_t)(3 + 8 * trip) * X_ROW_BYTES;
                uint8_t *ur = us + (uint32_t)(8 * trip) * 128u;
#pragma unroll
                for (int i0 = 0; i0 < 8; i0 += 4) {
                    f32x2 r01[7], r23[7];   // rows t-3 .. t+3 of the batch
#pragma unroll
                    for (int k = 0; k < 3; ++k) { r01[k] = h01[k]; r23[k] = h23[k]; }
#pragma unroll
                    for (int k = 0; k < 4; ++k) load_row(xr + (uint32_t)(i0 + k) * X_ROW_BYTES, r01[3 + k], r23[3 + k]);
                    f32x2 u01[4], u23[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) { u01[k] = fma2(w01[0], r01[3 + k], b01); u23[k] = fma2(w23[0], r23[3 + k], b23); }
#pragma unroll
                    for (int j = 1; j < 4; ++j) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) { u01[k] = fma2(w01[j], r01[3 + k - j], u01[k]); u23[k] = fma2(w23[j], r23[3 + k - j], u23[k]); }
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *(uint2 *)(ur + sw[i0 + k] + (uint32_t)(i0 + k) * 128u) =
                            make_uint2(pack_f16_sat(lo2(u01[k]), hi2(u01[k])), pack_f16_sat(lo2(u23[k]), hi2(u23[k])));
#pragma unroll
                    for (int k = 0; k < 3; ++k) { h01[k] = r01[4 + k]; h23[k] = r23[4 + k]; }
                }
            }
            fence_async_smem();  // make the generic-proxy writes of U visible to the tensor core
            __syncwarp();
            if (lane == 0) { mbar_arrive(BAR_XEMPTY(slot)); mbar_arrive_at(BAR_UFULL(st), 0); }
        }
        if (!ok && lane == 0) record_timeout();
    } else if (warp < 8) {
      reg_dec<40>();
      if (warp == 4) {
        // ================================================================ TMA loader
        const __nv_bfloat16 *x = (const __nv_bfloat16 *)f.x;
        const __nv_bfloat16 *cs_in = (const __nv_bfloat16 *)f.cs_in;
        bool ok = true;
        int b, ti;
        tile_first(b, ti);
        for (int it = 0; it < n_my_tiles; tile_next(it, b, ti), ++it) {
            const int slot = it % XS;
            ok = warp_wait_far(BAR_XEMPTY(slot), ((it / XS) & 1) ^ 1, spin, abort_flag);
            if (!ok) break;
            const int ts0 = ti * TILE + (int)rank * HALF;   // first token this CTA convolves
            const uint32_t dst = base + SMEM_X + slot * X_SLAB_BYTES;
            if (ts0 == 0 && cs_in != nullptr) {
                // first slab of a sequence with an incoming conv state: the three history rows come from
                // conv_state_in, so the slab is assembled from row copies
                const int hi_row = min(SLAB_ROWS, T + 3);
                // rows past the end of a short sequence are zeroed, as the tiled copy would have done (stale shared memory
                // could hold NaN patterns, and the gate arithmetic relies on a finite u for tokens that do not exist)
                for (int i = lane; i < (SLAB_ROWS - hi_row) * (int)(X_ROW_BYTES / 16); i += 32)
                    *(uint4 *)(smem + SMEM_X + slot * X_SLAB_BYTES + (uint32_t)hi_row * X_ROW_BYTES + (uint32_t)i * 16) = make_uint4(0, 0, 0, 0);
                __syncwarp();
                // of a narrower head only the channels that exist are copied (a whole row could run past the end of the tensor);
                // the rest of each row is zeroed for the same reason as the rows above
                const uint32_t row_bytes = (uint32_t)cvalid * 2;
                if (row_bytes < X_ROW_BYTES) {
                    const int per_row = (int)((X_ROW_BYTES - row_bytes) / 16);
                    for (int i = lane; i < hi_row * per_row; i += 32)
                        *(uint4 *)(smem + SMEM_X + slot * X_SLAB_BYTES + (uint32_t)(i / per_row) * X_ROW_BYTES + row_bytes + (uint32_t)(i % per_row) * 16) = make_uint4(0, 0, 0, 0);
                }
                __syncwarp();
                if (lane == 0) mbar_expect_tx(BAR_XFULL(slot), (uint32_t)hi_row * row_bytes);
                __syncwarp();
                for (int r = lane; r < hi_row; r += 32) {
                    const int t = r - 3;
                    const __nv_bfloat16 *src = t >= 0 ? x + ((size_t)b * T + t) * D + cbase
                                                      : cs_in + ((size_t)b * 3 + (3 + t)) * D + cbase;
                    bulk_g2s(dst + r * X_ROW_BYTES, src, row_bytes, BAR_XFULL(slot));
                }
            } else if (lane == 0) {
                // one tiled copy per slab: SLAB_ROWS token rows of this head starting three tokens early
                // (tokens before the sequence start and past its end read as zero)
                mbar_expect_tx(BAR_XFULL(slot), X_SLAB_BYTES);
                tma_load_3d(dst, &p.tm_x, cbase, ts0 - 3, b, BAR_XFULL(slot));
            }
            __syncwarp();
        }
        if (!ok && lane == 0) record_timeout();
      } else if ((warp == 5 || warp == 6) && rank == 0) {
        // ================================================================ MMA issuers of the pair: warp 5 the W_a products, warp 6 the W_x products
        // (one thread's issue stream is slow beside the busy warps of its scheduler; two streams on two schedulers keep the tensor pipe fed)
        const int gate = warp - 5;
        const uint32_t tm_w = gate ? TM_W_X : TM_W_A;
        constexpr uint32_t idesc = make_idesc_f16(256, TILE);
        bool ok = true;
        if (lane == 0) {
            ok = mbar_wait_cl(BAR_WREADY, 0, spin, abort_flag);
            for (int it = 0; it < n_my_tiles && ok; ++it) {
                const int st = it % US, bf = it & 1;
                ok = mbar_wait_cl(BAR_UFULL(st), (it / US) & 1, spin, abort_flag);
                if (!ok) break;
                ok = mbar_wait_cl(BAR_ACCEMPTY(bf), ((it >> 1) & 1) ^ 1, spin, abort_flag);
                if (!ok) break;
                tc_fence_after();
                // the start-address field of the descriptor counts 16-byte units; the same offset addresses each CTA's own stage
                const uint64_t bd0 = make_desc_sw128(base + SMEM_U + st * U_STAGE_BYTES);
                const uint32_t acc = tmem + tm_acc(bf, gate);
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    const uint64_t bd = bd0 + (uint64_t)(((ks >> 2) * U_KBLOCK_BYTES + (ks & 3) * 32) >> 4);
                    mma_ts2(acc, tmem + tm_w + ks * 8, bd, idesc, ks > 0);
                }
                tc_commit2(BAR_UEMPTY(st), (uint16_t)3);
                tc_commit2(BAR_ACCFULL(bf), (uint16_t)3);
            }
            if (!ok) record_timeout();
        }
        __syncwarp();
      }
    } else if (warp < 16) {
        // ================================================================ gate warps
        reg_inc<112>();
        const int q = warp & 3, g = (warp - 8) >> 2;     // lane quarter; tokens [32 g, 32 g + 32) of every tile, convolved by CTA g
        const int hc = (int)rank * CH + q * 32 + lane;   // channel within the head
        const int d = cbase + hc;                        // global channel
        const bool exists = hc < cvalid;                 // uniform over the warp (widths are multiples of 32)
        // per-channel constants; s = c softplus(-Lambda) with libm-grade log1p/exp (Appendix A)
        const float lam = exists ? f.lambda[d] : 0.0f;
        const float zl = -lam;
        const float s = f.c * (zl > 0.0f ? zl + log1pf(expf(-zl)) : log1pf(expf(zl)));
        const f32x2 s2 = pack2(s, s);
        const float ba_c = exists ? f.b_a[d] : 0.0f, bx_c = exists ? f.b_x[d] : 0.0f;
        const f32x2 hba2 = pack2(0.5f * ba_c, 0.5f * ba_c), hbx2 = pack2(0.5f * bx_c, 0.5f * bx_c);
        const bool poly = __all_sync(0xffffffffu, s <= S_POLY);
        // u[row][channel] in the swizzled U tile of CTA g, one offset per row phase (row & 7)
        const bool remote = (uint32_t)g != rank;
        const uint32_t u_cta = remote ? map_to_cta(base, (uint32_t)g) : base;
        uint32_t u_off[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            u_off[j] = u_cta + SMEM_U + (uint32_t)(hc >> 6) * U_KBLOCK_BYTES + ((((uint32_t)(hc & 63) >> 3) ^ (uint32_t)j) << 4) + (uint32_t)(hc & 7) * 2;
        const uint32_t tm_lane = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * HALF);
        float2 *agg_mine = (float2 *)(smem + SMEM_AGG) + g * CH + q * 32 + lane;
        bool ok = true;
        int b, ti;
        tile_first(b, ti);
        for (int it = 0; it < n_my_tiles; tile_next(it, b, ti), ++it) {
            const int st = it % US, bf = it & 1;
            const int nvh = T - ti * TILE - g * HALF;    // tokens of this warp's half tile that exist (may be <= 0 or >= HALF)
            ok = warp_wait_cl(BAR_ACCFULL(bf), (it >> 1) & 1, spin, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t ta = tm_lane + tm_acc(bf, 0), tx = tm_lane + tm_acc(bf, 1);
            const uint32_t ust = (uint32_t)st * U_STAGE_BYTES;
            float c = 1.0f, h = 0.0f;   // running product of a_t and state from zero over this half tile
            // Sixteen tokens (eight pairs of adjacent tokens) at a time: (z_a, z_x) from tensor memory and u from the U tile ->
            // gates -> (a_t, v_t) -> scan from zero state -> column t becomes (prod_{s<=t} a_s, h_t from zero), written back
            // in place.  Eight independent chains per instruction keep the pipes busy in spite of in-order issue; the loop
            // over the two batches stays rolled to keep the code small.
#pragma unroll 1
            for (int bt = 0; bt < 2; ++bt) {
                f32x2 ZA[8], ZX[8];
                float u[16];
                tmem_ld16(ta + 16 * bt, ZA);
                tmem_ld16(tx + 16 * bt, ZX);
                const uint32_t row0 = ust + (uint32_t)(16 * bt) * 128u;
                if (remote) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) u[e] = f16_bits_to_f32((uint16_t)ld_cluster_u16(u_off[e & 7] + row0 + (uint32_t)e * 128u));
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) u[e] = f16_bits_to_f32((uint16_t)ld_shared_u16(u_off[e & 7] + row0 + (uint32_t)e * 128u));
                }
                tmem_ld_wait();
                if (nvh < HALF) {
                    // ragged tail: a token that does not exist gets z_a = -inf-like, which the gate arithmetic turns into
                    // a_t = 1, v_t = 0 exactly (r = 0, so log a = 0 and sqrt(1 - a^2) = 0; its u is finite), i.e. it holds the state
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        ZA[j] = pack2(16 * bt + 2 * j < nvh ? lo2(ZA[j]) : -1e30f, 16 * bt + 2 * j + 1 < nvh ? hi2(ZA[j]) : -1e30f);
                }
                if (poly) gate_group<true, 8>(ZA, ZX, u, hba2, hbx2, s2);
                else gate_group<false, 8>(ZA, ZX, u, hba2, hbx2, s2);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float a0 = lo2(ZA[i]), a1 = hi2(ZA[i]);
                    const float c0 = c * a0, h0 = fmaf(a0, h, lo2(ZX[i]));
                    c = c0 * a1; h = fmaf(a1, h0, hi2(ZX[i]));
                    ZA[i] = pack2(c0, c); ZX[i] = pack2(h0, h);
                }
                tmem_st16(ta + 16 * bt, ZA);
                tmem_st16(tx + 16 * bt, ZX);
            }
            agg_mine[bf * 2 * CH] = make_float2(c, h);   // the half tile as one step: h_out = c h_in + h
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(BAR_GDONE(bf, q));                  // this warp's half of the tile is in tensor memory
                mbar_arrive_at(BAR_UEMPTY(st), (uint32_t)g);    // done reading u from CTA g's stage
            }
        }
        if (!ok && lane == 0) record_timeout();
    } else {
        // ================================================================ scan warps
        reg_inc<152>();
        const int q = warp & 3;
        const int c_own = q * 32 + lane;                 // channel within the CTA
        const int d = cbase + (int)rank * CH + c_own;    // global channel
        const bool exists = (int)rank * CH + c_own < cvalid;   // uniform over the warp; a warp of channel slots that do not exist
                                                                // keeps the barriers going but reads and writes no global memory
        const uint32_t tm_lane = tmem + ((uint32_t)(q * 32) << 16);
        const uint32_t y_warp_off = SMEM_Y + (uint32_t)q * 2 * Y_BUF_BYTES;
        const float2 *agg_s = (const float2 *)(smem + SMEM_AGG) + c_own;
        const __nv_bfloat16 *x = (const __nv_bfloat16 *)f.x;
        const __nv_bfloat16 *cs_in = (const __nv_bfloat16 *)f.cs_in;
        float h_prev_own = 0.0f;  // state at the end of this pair's previous tile
        float P_prev_own = 1.0f;  // prod of a_t from the start of the sequence to the end of this pair's previous tile
        constexpr bool merged = MERGED;
        bool ok = true;
        int b, ti;
        tile_first(b, ti);
        for (int it = 0; it < n_my_tiles; tile_next(it, b, ti), ++it) {
            const bool shared = it < n_shared;
            const int gidx = (b - B_whole) * p.tps + ti;   // index of the tile's carry record (shared tiles only)
            const int t0 = ti * TILE;
            const int bf = it & 1;
            const uint32_t y_off = y_warp_off + (uint32_t)bf * Y_BUF_BYTES;
            if constexpr (merged) {
                // The warp's 64 x 32 block of the gate branch is fetched into the y staging buffer of this tile (free once
                // the store of two tiles ago has read it) while the gate warps still work; y then overwrites it in place.
                if (lane == 0 && exists) {
                    bulk_wait_read1();
                    mbar_expect_tx(BAR_BRANCH(q), Y_BUF_BYTES);
                    tma_load_3d(base + y_off, &p.tm_g, cbase + (int)rank * CH + q * 32, t0, b, BAR_BRANCH(q));
                }
                __syncwarp();
            }
            ok = warp_wait(BAR_GDONE(bf, q), (it >> 1) & 1, spin, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // the two half tiles as steps h_out = e.x h_in + e.y
            const float2 e0 = agg_s[(bf * 2 + 0) * CH], e1 = agg_s[(bf * 2 + 1) * CH];
            // ---- incoming state of the tile: the state this pair reached at the end of its previous tile, or h0 near the
            //      start of a sequence, advanced by the aggregates that the other pairs published for the tiles in between
            float h, P;
            if (!shared) {
                h = ti == 0 ? (f.h0 && exists ? f.h0[(size_t)b * D + d] : 0.0f) : h_prev_own;
                P = ti == 0 ? 1.0f : P_prev_own;
            } else {
                // publish the tile's aggregate before waiting for anyone
                uint4 rec;
                rec.x = __float_as_uint(e0.x * e1.x); rec.y = p.tag; rec.z = __float_as_uint(fmaf(e1.x, e0.y, e1.y)); rec.w = p.tag;
                uint4 *dst = p.agg + ((size_t)group * p.tiles_total + gidx) * CH + c_own;
                asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(rec.x), "r"(rec.y), "r"(rec.z), "r"(rec.w) : "memory");
                int nback;
                if (ti < S) { h = f.h0 && exists ? f.h0[(size_t)b * D + d] : 0.0f; P = 1.0f; nback = ti; }
                else { h = h_prev_own; P = P_prev_own; nback = S - 1; }
                // The records are taken oldest first, up to eight at a time: all of a batch are requested at once, then polled
                // until every lane sees this call's tag in both halves of each record (8-byte words are written atomically).
                const uint4 *src = p.agg + ((size_t)group * p.tiles_total + gidx) * CH + c_own;
                for (int jb = nback; jb > 0 && ok; jb -= LOOKBACK_BATCH) {
                    const int cnt = jb < LOOKBACK_BATCH ? jb : LOOKBACK_BATCH;   // records jb, jb - 1, ..., jb - cnt + 1 tiles back
                    uint4 r[LOOKBACK_BATCH];
                    uint64_t tstart = 0;
                    for (uint32_t npoll = 0;; ++npoll) {
                        bool ready = true;
#pragma unroll
                        for (int k = 0; k < LOOKBACK_BATCH; ++k) {
                            if (k < cnt) {
                                const uint4 *sj = src - (size_t)(jb - k) * CH;
                                asm volatile("ld.volatile.global.v4.b32 {%0, %1, %2, %3}, [%4];"
                                             : "=r"(r[k].x), "=r"(r[k].y), "=r"(r[k].z), "=r"(r[k].w) : "l"(sj) : "memory");
                            }
                        }
#pragma unroll
                        for (int k = 0; k < LOOKBACK_BATCH; ++k)
                            if (k < cnt) ready = ready && r[k].y == p.tag_wait && r[k].w == p.tag_wait;
                        if (__all_sync(0xffffffffu, ready)) break;
                        if ((npoll & 15u) == 15u) {
                            const uint64_t tnow = gtimer();
                            if (tstart == 0) tstart = tnow;
                            if (*abort_flag || tnow - tstart > spin) { ok = false; break; }
                        }
                        __nanosleep(32);
                    }
                    ok = __all_sync(0xffffffffu, ok);
                    if (ok) {
#pragma unroll
                        for (int k = 0; k < LOOKBACK_BATCH; ++k)
                            if (k < cnt) { h = fmaf(__uint_as_float(r[k].x), h, __uint_as_float(r[k].z)); P *= __uint_as_float(r[k].x); }
                    }
                }
                if (!ok) break;
            }
            const float h_mid = fmaf(e0.x, h, e0.y);      // state after the first half tile
            h_prev_own = fmaf(e1.x, h_mid, e1.y);         // state after the tile
            P_prev_own = P * (e0.x * e1.x);
            // ---- the y block written two tiles ago must have been read out by its tiled store
            if (lane == 0) bulk_wait_read1();
            __syncwarp();
            // ---- y_t = h_t = (h_t from zero) + (prod a up to t) h_in  (Eq. 4 unrolled over the half tile), 16 tokens at a time
            uint16_t *y_s = (uint16_t *)(smem + y_off) + lane;   // this thread's column of the warp's y block [64 tokens][32 channels]
            // The whole tile is pulled into registers and the accumulator buffer handed back before any arithmetic: the buffer's
            // round trip (MMA -> gate warps -> here -> MMA) is what paces the kernel.
            float C[TILE], H[TILE];
            const uint32_t tc = tm_lane + tm_acc(bf, 0), th = tm_lane + tm_acc(bf, 1);
#pragma unroll
            for (int c0 = 0; c0 < TILE; c0 += 16) { tmem_ld16f(tc + c0, C + c0); tmem_ld16f(th + c0, H + c0); }
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_at(BAR_ACCEMPTY(bf), 0);
            if constexpr (merged) {
                // merged output of the recurrent block (Section 2.3): y_t = h_t GeLU(branch_t); the state is not touched
                if (exists) {
                    ok = warp_wait(BAR_BRANCH(q), it & 1, spin, abort_flag);
                    if (!ok) break;
                }
#pragma unroll
                for (int j = 0; j < TILE; j += 2) {
                    const float hb = j < HALF ? h : h_mid;
                    const float g0 = __uint_as_float((uint32_t)y_s[j * 32] << 16), g1 = __uint_as_float((uint32_t)y_s[(j + 1) * 32] << 16);
                    const f32x2 ym = gelu_times2(fma2(pack2(C[j], C[j + 1]), pack2(hb, hb), pack2(H[j], H[j + 1])), g0, g1);
                    const __nv_bfloat162 o = __floats2bfloat162_rn(lo2(ym), hi2(ym));
                    const uint32_t ow = *(const uint32_t *)&o;
                    y_s[j * 32] = (uint16_t)(ow & 0xFFFFu);
                    y_s[(j + 1) * 32] = (uint16_t)(ow >> 16);
                }
            } else {
#pragma unroll
                for (int j = 0; j < TILE; j += 2) {
                    const float hb = j < HALF ? h : h_mid;
                    const float y0 = fmaf(C[j], hb, H[j]), y1 = fmaf(C[j + 1], hb, H[j + 1]);
                    const __nv_bfloat162 o = __floats2bfloat162_rn(y0, y1);
                    const uint32_t ow = *(const uint32_t *)&o;
                    y_s[j * 32] = (uint16_t)(ow & 0xFFFFu);             // row of the warp's block: 32 channels x 2 bytes
                    y_s[(j + 1) * 32] = (uint16_t)(ow >> 16);
                }
            }
            fence_async_smem();   // y rows become visible to the bulk-copy engine
            __syncwarp();
            if (lane == 0 && exists) {
                // the warp's 64 tokens x 32 channels go out as one tiled store; rows at or beyond T are clipped
                tma_store_3d(&p.tm_y, cbase + (int)rank * CH + q * 32, t0, b, base + y_off);
                bulk_commit();
            }
            if (ti == p.tps - 1 && exists) {
                // end of a sequence: h_T (unrounded state) and the last three raw inputs, bit-exact
                f.h_T[(size_t)b * D + d] = h_prev_own;
                if (f.a_prod) f.a_prod[(size_t)b * D + d] = P_prev_own;
                __nv_bfloat16 keep[3];
#pragma unroll
                for (int kk = 0; kk < 3; ++kk) {
                    const int t = T - 3 + kk;
                    keep[kk] = t >= 0 ? x[((size_t)b * T + t) * D + d]
                                      : (cs_in ? cs_in[((size_t)b * 3 + (3 + t)) * D + d] : __float2bfloat16_rn(0.0f));
                }
                __nv_bfloat16 *cs_out = (__nv_bfloat16 *)f.cs_out;
#pragma unroll
                for (int kk = 0; kk < 3; ++kk) cs_out[((size_t)b * 3 + kk) * D + d] = keep[kk];
            }
        }
        if (lane == 0) bulk_wait0();
        ok = __all_sync(0xffffffffu, ok);
        if (!ok && lane == 0) record_timeout();
    }

    // ---- teardown: every role falls through to here, also after a timeout
    if (*abort_flag) {
        // let copies and MMAs in flight land before shared and tensor memory are given back
        const uint64_t tw = gtimer();
        while (gtimer() - tw < 50000ull) __nanosleep(1000);
    }
    tc_fence_before();
    cluster_arrive();   // neither CTA leaves while its peer may still read its shared memory or arrive on its barriers
    cluster_wait();
    if (warp == 5) tmem_dealloc2(tmem, 512);
}

// Per-device launch facts, looked up once per device with that device current.
struct DeviceInfo {
    bool ready = false;
    int sms = 148;
    int max_pairs = 70;   // CTA pairs that can be resident at once
};
std::mutex g_dev_mutex;
DeviceInfo g_dev[64];

cudaError_t device_info(DeviceInfo *out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DeviceInfo &di = g_dev[dev];
    if (!di.ready) {
        // opt in to the large dynamic shared memory once per device (function attributes are per context)
        e = cudaFuncSetAttribute(sm100_prefill_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(sm100_prefill_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) di.sms = n;
        cudaLaunchConfig_t q{};
        q.gridDim = dim3(2 * di.sms); q.blockDim = dim3(NUM_THREADS); q.dynamicSmemBytes = SMEM_ALLOC;
        int np = 0;
        // a pair needs two free SMs of one cluster-capable group, so fewer than sms / 2 pairs may fit
        di.max_pairs = (cudaOccupancyMaxActiveClusters(&np, sm100_prefill_kernel<false>, &q) == cudaSuccess && np > 0) ? np : di.sms / 2 - 4;
        di.ready = true;
    }
    *out = di;
    return cudaSuccess;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (the library does not link libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            ptr = nullptr;
        return (EncodeTiledFn)ptr;
    }();
    return fn;
}

// Tensor map of a bf16 [B][T][D] activation tensor with a box of box_t token rows x box_c channels.
bool make_activation_map(CUtensorMap *tm, const void *ptr, int B, int T, int D, int box_c, int box_t) {
    return encode_bf16_map_3d(tm, ptr, (uint64_t)D, (uint64_t)T, (uint64_t)B, (uint32_t)box_c, (uint32_t)box_t, false);
}

std::atomic<uint32_t> g_call_counter{0};

uint32_t next_tag() {
    static const uint32_t salt = (uint32_t)std::chrono::steady_clock::now().time_since_epoch().count() * 2654435761u;
    uint32_t t = salt + 0x9E3779B9u * (g_call_counter.fetch_add(1) + 1u);
    return t == 0 ? 1u : t;
}

}  // namespace

unsigned long long g_spin_limit_ns = 2000000000ull;  // bounded waits give up after this long

bool encode_map16_3d(CUtensorMap *tm, const void *ptr, const uint64_t dims[3], const uint64_t strides_bytes[2], const uint32_t box[3],
                     bool swizzle128) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (enc == nullptr) return false;
    const cuuint64_t d[3] = {dims[0], dims[1], dims[2]};
    const cuuint64_t st[2] = {strides_bytes[0], strides_bytes[1]};
    const cuuint32_t bx[3] = {box[0], box[1], box[2]};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), d, st, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_bf16_map_3d(CUtensorMap *tm, const void *ptr, uint64_t d0, uint64_t d1, uint64_t d2, uint32_t box0, uint32_t box1,
                        bool swizzle128) {
    const uint64_t dims[3] = {d0, d1, d2}, strides[2] = {d0 * 2, d0 * d1 * 2};
    const uint32_t box[3] = {box0, box1, 1};
    return encode_map16_3d(tm, ptr, dims, strides, box, swizzle128);
}

namespace {
// layer heads per kernel "head" (a group of consecutive heads sharing 256 channel slots), and the number of such groups
inline int heads_per_group(int D, int H) { return DH / (D / H); }
inline int kernel_heads(int D, int H) { const int k = heads_per_group(D, H); return (H + k - 1) / k; }
}  // namespace
// Head width: any multiple of 32 up to 256.  k = 256 / width (rounded down) consecutive heads share the kernel's 256 channel
// slots; slots beyond k width (and beyond the layer's last head) do not exist: zero weights and taps, never loaded per
// element or stored.
bool sm100_prefill_supported(int B, int T, int D, int H, int io) {
    if (io != RGLRU_BF16 || B <= 0 || T <= 0 || H <= 0 || D % H != 0) return false;
    const int dh = D / H;
    return dh <= DH && dh % 32 == 0;
}

namespace {
inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }
// Pairs that share a head's time axis: as many as fit beside the other heads, at most MAX_S.  The host-only workspace
// size has to agree with the launch, so both count with at most MAX_PAIRS pairs whatever the device reports.
constexpr int MAX_PAIRS = 74;
inline int pairs_per_head(int H, int pairs) {
    if (pairs > MAX_PAIRS) pairs = MAX_PAIRS;
    int S = pairs / H;
    return S < 1 ? 1 : (S > MAX_S ? MAX_S : S);
}
// Carry records exist for the sequences that are split in time: B mod S of them, at most S - 1 with S <= pairs_per_head(H, MAX_PAIRS).
// Record (sequence slot, tile, half-head, channel) is indexed as [half-head][slot * tps + tile][channel].
inline int record_slots(int B, int H) {
    const int most = pairs_per_head(H, MAX_PAIRS) - 1;
    return B < most ? B : most;
}
size_t agg_bytes(int B, int T, int H) {
    const size_t tps = (T + TILE - 1) / TILE;
    return up256((size_t)H * 2 * record_slots(B, H) * tps * CH * sizeof(uint4));
}
inline bool ranges_overlap(const void *a, const void *b, size_t n) {
    if (!a || !b) return false;
    const uintptr_t pa = (uintptr_t)a, pb = (uintptr_t)b;
    return pa < pb + n && pb < pa + n;
}
}  // namespace

// Workspace body: aggregate records | private copy of h0 | private copy of conv_state_in.
// The copies are used only when the caller's state outputs alias the state inputs: CTAs of
// different tiles and of the two halves of a head read the incoming state at unrelated times,
// so an in-place update must not be visible to them.
size_t sm100_prefill_workspace_bytes(int B, int T, int D, int H) {
    H = kernel_heads(D, H);   // the kernel's unit: a 256-channel group of heads, or one head of another width
    return agg_bytes(B, T, H) + up256((size_t)B * D * sizeof(float)) + up256((size_t)B * 3 * D * sizeof(__nv_bfloat16));
}

cudaError_t sm100_prefill(const FwdArgs &a, void *ws_body, size_t ws_body_bytes, cudaStream_t st) {
    cudaError_t e;
    DeviceInfo di;
    if ((e = device_info(&di)) != cudaSuccess) return e;
    Sm100Args p;
    if (!make_activation_map(&p.tm_x, a.x, a.B, a.T, a.D, DH, SLAB_ROWS) || !make_activation_map(&p.tm_y, a.y, a.B, a.T, a.D, 32, TILE))
        return cudaErrorNotSupported;
    if (a.gate_branch) {
        if (!make_activation_map(&p.tm_g, a.gate_branch, a.B, a.T, a.D, 32, TILE)) return cudaErrorNotSupported;
    } else {
        p.tm_g = p.tm_y;   // never used by the kernel
    }
    p.f = a;
    const int G = kernel_heads(a.D, a.H);   // 256-channel groups of heads, or heads of another width: the kernel's "heads"
    p.f.H = G;
    p.dh = a.D / a.H;
    p.hstride = heads_per_group(a.D, a.H) * p.dh;
    p.cvalid = p.hstride;
    p.tps = (a.T + TILE - 1) / TILE;
    const int pairs = di.max_pairs < di.sms / 2 ? di.max_pairs : di.sms / 2;
    int S = pairs_per_head(G, pairs);
    if (S > a.B * p.tps) S = a.B * p.tps;
    p.S = S;
    p.tiles_total = record_slots(a.B, G) * p.tps;
    p.tag = next_tag();
    p.tag_wait = (a.flags & RGLRU_FLAG_TEST_CARRY_NEVER_ARRIVES) ? ~p.tag : p.tag;
    p.agg = (uint4 *)ws_body;
    p.spin_ns = g_spin_limit_ns;
    if (ws_body_bytes < sm100_prefill_workspace_bytes(a.B, a.T, a.D, a.H)) return cudaErrorInvalidValue;
    const size_t h_bytes = (size_t)a.B * a.D * sizeof(float), cs_bytes = (size_t)a.B * 3 * a.D * sizeof(__nv_bfloat16);
    char *h0_copy = (char *)ws_body + agg_bytes(a.B, a.T, G), *cs_copy = h0_copy + up256(h_bytes);
    if (ranges_overlap(a.h0, a.h_T, h_bytes)) {
        if ((e = cudaMemcpyAsync(h0_copy, a.h0, h_bytes, cudaMemcpyDeviceToDevice, st)) != cudaSuccess) return e;
        p.f.h0 = (const float *)h0_copy;
    }
    if (ranges_overlap(a.cs_in, a.cs_out, cs_bytes)) {
        if ((e = cudaMemcpyAsync(cs_copy, a.cs_in, cs_bytes, cudaMemcpyDeviceToDevice, st)) != cudaSuccess) return e;
        p.f.cs_in = cs_copy;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * G * S); cfg.blockDim = dim3(NUM_THREADS); cfg.dynamicSmemBytes = SMEM_ALLOC; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;   // pairs wait on one another's aggregates: they must all be resident
    attr[0].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = (S > 1 && a.B % S != 0) ? 1 : 0;
    return a.gate_branch ? cudaLaunchKernelEx(&cfg, sm100_prefill_kernel<true>, p) : cudaLaunchKernelEx(&cfg, sm100_prefill_kernel<false>, p);
}

}  // namespace rglru
