// sm_100a fused prefill for the RG-LRU temporal core (bf16 io, head width 256).
//
// One persistent CTA per SM owns HALF a head (128 channels): its 2 x 128 rows of W_a and W_x stay
// resident in tensor memory as the A operand of tcgen05.mma for the whole launch.  The CTA walks
// tiles of 128 tokens:
//   TMA warp       x rows of the whole head (the gates need all 256 input channels) -> shared memory, tiled copies
//   conv warps     causal width-4 depthwise conv in fp32 -> fp16 tile U[128 tokens][256 ch] in the
//                  K-major 128B-swizzled layout tcgen05.mma reads as its B operand
//   MMA warps      Z_a^T = W_a U^T (one warp) and Z_x^T = W_x U^T (another): channels on TMEM lanes, time along
//                  TMEM columns, one N = 128 instruction per K step
//   epilogue warps tcgen05.ld (time runs along registers, so the scan needs no shuffles), gates,
//                  log-space decay, the linear recurrence in fp32, y through a per-warp tiled store
// x is read from HBM once per head (the two half-head CTAs share it through L2), y is written once;
// u, r, i, a never leave the SM.
//
// Time is split across CTAs so that every SM has work even for a single long sequence: sequences that
// cannot be dealt out whole go to the S CTAs of a half-head tile by tile, round-robin.  Such a tile first folds itself to the aggregate
// (prod a_t, h_end from zero state), publishes it, and obtains its incoming state from its own
// previous tile plus the S-1 aggregates published by the other CTAs (decoupled look-back); only
// then does it run the real scan and write y.  Waits on other CTAs are bounded and end in
// RGLRU_ERR_TIMEOUT; the launch is cooperative so that all CTAs are co-resident.
#include <cooperative_groups.h>
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <chrono>
#include <type_traits>

#include "rglru_internal.h"
#include "sm100_ptx.cuh"
#include "sm100_gates.cuh"

namespace rglru {
namespace {

constexpr int DH = 256;            // head width handled by this kernel
constexpr int CH = 128;            // channels per CTA (half a head)
constexpr int TILE_N = 128;        // tokens per MMA tile
constexpr int SLAB = 32;           // tokens per TMA slab
constexpr int SLAB_ROWS = SLAB + 3;
constexpr int XS = 3;              // x slab ring depth
constexpr int US = 2;              // U tile stages
constexpr int NUM_THREADS = 512;
constexpr int EPI_TOK = 64;        // tokens per epilogue warp
constexpr int MAX_S = 8;           // at most this many CTAs share one half-head's time axis
constexpr uint32_t U_STAGE_BYTES = TILE_N * DH * 2;       // 65536
constexpr uint32_t U_KBLOCK_BYTES = TILE_N * 128;          // 16384: one 64-channel K block
constexpr uint32_t X_ROW_BYTES = DH * 2;                   // 512
constexpr uint32_t X_SLAB_BYTES = SLAB_ROWS * X_ROW_BYTES; // 17920
constexpr uint32_t SMEM_U = 0;
constexpr uint32_t SMEM_X = SMEM_U + US * U_STAGE_BYTES;
constexpr uint32_t Y_WARP_BYTES = EPI_TOK * 32 * 2;        // 4096: one epilogue warp's 64 tokens x 32 channels
constexpr uint32_t SMEM_Y = SMEM_X + XS * X_SLAB_BYTES;    // bf16 y_s[8 warps][64][32], staged for tiled stores
constexpr uint32_t SMEM_AGG = SMEM_Y + 8 * Y_WARP_BYTES;   // float2 agg_s[2 tile parity][2 halves][4][32]
constexpr uint32_t SMEM_BAR = SMEM_AGG + 2 * 2 * 4 * 32 * 8;
constexpr int NUM_BARS = 2 * XS + 2 * US + 4 + 8 + 1;
constexpr uint32_t SMEM_MISC = SMEM_BAR + NUM_BARS * 8;    // tmem base, abort flag
constexpr uint32_t SMEM_TOTAL = SMEM_MISC + 16;
constexpr uint32_t SMEM_ALLOC = SMEM_TOTAL + 1024;         // slack for 1024-byte alignment

// TMEM columns
constexpr uint32_t TM_ACC_A = 0, TM_ACC_X = 128, TM_W_A = 256, TM_W_X = 384;


struct Sm100Args {
    // x as [B][T][D] with a box of SLAB_ROWS token rows x one head; y with a box of EPI_TOK rows x 32 channels
    alignas(64) CUtensorMap tm_x;
    alignas(64) CUtensorMap tm_y;
    FwdArgs f;
    int S;             // CTAs per half-head (time split factor)
    int tps;           // tiles per sequence
    int tiles_total;   // B * tps
    uint32_t tag;      // validity tag of this call's aggregate records
    uint4 *agg;        // [H*2][tiles_total][128] records {P, tag, h_loc, tag}
    unsigned long long spin_ns;
};

using namespace ptx;

__device__ __forceinline__ void record_timeout(uint32_t *status, volatile int *abort_flag) {
    *abort_flag = 1;
    atomicExch(status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT);
}

__global__ void __launch_bounds__(NUM_THREADS, 1) sm100_prefill_kernel(const __grid_constant__ Sm100Args p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    const uint32_t bar0 = base + SMEM_BAR;
    // barrier indices
    auto BAR_XFULL = [&](int s) { return bar0 + 8u * s; };
    auto BAR_XEMPTY = [&](int s) { return bar0 + 8u * (XS + s); };
    auto BAR_UFULL = [&](int s) { return bar0 + 8u * (2 * XS + s); };
    auto BAR_UEMPTY = [&](int s) { return bar0 + 8u * (2 * XS + US + s); };
    auto BAR_ACCFULL = [&](int k) { return bar0 + 8u * (2 * XS + 2 * US + k); };       // accumulators of token half k
    auto BAR_ACCEMPTY = [&](int k) { return bar0 + 8u * (2 * XS + 2 * US + 2 + k); };
    auto BAR_AGG = [&](int q, int k) { return bar0 + 8u * (2 * XS + 2 * US + 4 + q * 2 + k); };  // fold of half k, channel group q
    const uint32_t BAR_WREADY = bar0 + 8u * (2 * XS + 2 * US + 12);   // gate weights are in tensor memory
    uint32_t *tmem_base_s = (uint32_t *)(smem + SMEM_MISC);
    volatile int *abort_flag = (volatile int *)(smem + SMEM_MISC + 4);
    float2 *agg_s = (float2 *)(smem + SMEM_AGG);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const FwdArgs &f = p.f;
    const int T = f.T, D = f.D, S = p.S;
    const int group = blockIdx.x / S, kcta = blockIdx.x % S;  // group = head * 2 + half
    const int head = group >> 1, half = group & 1;
    // Work of this CTA.  Sequences are dealt out whole where that keeps the S CTAs of the half-head balanced: CTA kcta
    // gets sequences kcta, kcta + S, ... of the first (B / S) * S ones and walks each from start to end, so a tile's
    // incoming state is simply the state the CTA itself reached ("local" tiles: no record, no look-back).  The B % S
    // sequences left over are split in time, tile g of them going to CTA g % S ("shared" tiles, decoupled look-back).
    // Shared tiles come first, so that the S CTAs pass through them in step.
    const int B_whole = (f.B / S) * S, shared_tiles = (f.B - B_whole) * p.tps;
    const int n_shared = kcta < shared_tiles ? (shared_tiles - kcta + S - 1) / S : 0;
    const int n_my_tiles = n_shared + (B_whole / S) * p.tps;
    // The CTA's tiles in order: tile_first gives (sequence b, tile ti within it) of tile 0, tile_next steps from tile
    // `it` to tile `it + 1`; tile `it` is a shared one when it < n_shared.
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
        for (int s = 0; s < US; ++s) { mbar_init(BAR_UFULL(s), 4); mbar_init(BAR_UEMPTY(s), 10); }
        mbar_init(BAR_ACCFULL(0), 2); mbar_init(BAR_ACCEMPTY(0), 8);
        for (int q = 0; q < 4; ++q) { mbar_init(BAR_AGG(q, 0), 1); mbar_init(BAR_AGG(q, 1), 1); }
        mbar_init(BAR_WREADY, 8);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) { tmem_alloc(smem_u32(tmem_base_s), 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_base_s;

    // Gate weights of this half-head into tensor memory: lane = output channel, 32-bit column j holds
    // input channels 2j (low half) and 2j+1 (high half).  The tensor core multiplies them with the conv output
    // u, which is kept in fp16 (11 significant bits instead of bf16's 8, because u also enters i_t * u_t of
    // Eq. 4 directly), and both operands of one MMA must have one type: the bf16 weights are converted to
    // fp16 here, which is exact for every weight of magnitude within [2^-14, 65504] and rounds tinier ones
    // to a multiple of 2^-24.
    if (warp >= 8) {
        const int q = warp & 3, g = (warp - 8) >> 2;  // g = 0: W_a, 1: W_x
        const __nv_bfloat16 *W = (const __nv_bfloat16 *)(g ? f.W_x : f.W_a);
        const uint4 *row = (const uint4 *)(W + ((size_t)head * DH + half * CH + q * 32 + lane) * DH);
        const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (g ? TM_W_X : TM_W_A);
        auto cvt2 = [](uint32_t w) { return pack_f16_sat(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u)); };
#pragma unroll 4
        for (int c = 0; c < 16; ++c) {
            uint4 lo = __ldg(row + 2 * c), hi = __ldg(row + 2 * c + 1);
            lo.x = cvt2(lo.x); lo.y = cvt2(lo.y); lo.z = cvt2(lo.z); lo.w = cvt2(lo.w);
            hi.x = cvt2(hi.x); hi.y = cvt2(hi.y); hi.z = cvt2(hi.z); hi.w = cvt2(hi.w);
            tmem_st8(taddr + c * 8, lo, hi);
        }
        tmem_st_wait();
        // only the MMA issuers wait for the weights: loads and the conv of the first tiles run meanwhile
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR_WREADY);
    }

    // Register budget per warpgroup (the four warps of a group execute the same setmaxnreg):
    // conv producers 72, loader / MMA issuer / idle 40, epilogue 200.
    if (warp < 4) {
        // ================================================================ conv producers
        reg_dec<72>();
        const int pblk = warp;                       // K block = 64 channels of the head
        const int l16 = lane & 15, tg = lane >> 4;   // 4-channel chunk, token group of 16
        const int hc = pblk * 64 + l16 * 4;          // channel within the head
        const __nv_bfloat16 *cw = (const __nv_bfloat16 *)f.conv_w;
        f32x2 w01[4], w23[4], b01, b23;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const __nv_bfloat16 *wp = cw + (size_t)j * D + head * DH + hc;
            w01[j] = pack2(__bfloat162float(wp[0]), __bfloat162float(wp[1]));
            w23[j] = pack2(__bfloat162float(wp[2]), __bfloat162float(wp[3]));
        }
        if (f.conv_b) {
            const float *bp = f.conv_b + head * DH + hc;
            b01 = pack2(bp[0], bp[1]); b23 = pack2(bp[2], bp[3]);
        } else { b01 = pack2(0.f, 0.f); b23 = b01; }
        const uint32_t x_thread_off = (uint32_t)hc * 2;
        const uint32_t u_chunk = (uint32_t)(l16 >> 1), u_half = (uint32_t)(l16 & 1) * 8;
        // Token tt of a tile is stored in row perm(tt) of the U tile (= accumulator column perm(tt)):
        // within each group of 64 tokens, tokens j and j + 32 sit in adjacent rows 2j and 2j + 1, so that
        // the epilogue finds them in one register pair and can run the two halves of its 64 tokens as
        // the two lanes of packed fp32x2 arithmetic.
        int slab_n = 0;
        bool ok = true;
        int b, ti;
        tile_first(b, ti);
        for (int it = 0; it < n_my_tiles && ok; tile_next(it, b, ti), ++it) {
            const int t0 = ti * TILE_N;
            const int st = it % US;
            ok = warp_wait(BAR_UEMPTY(st), ((it / US) & 1) ^ 1, spin, abort_flag);
            if (!ok) break;
            const uint32_t u_base = SMEM_U + st * U_STAGE_BYTES + pblk * U_KBLOCK_BYTES + u_half;  // offset from smem
            const int nslab = min(TILE_N / SLAB, (T - t0 + SLAB - 1) / SLAB);
            for (int s = 0; s < nslab; ++s, ++slab_n) {
                const int slot = slab_n % XS;
                ok = warp_wait(BAR_XFULL(slot), (slab_n / XS) & 1, spin, abort_flag);
                if (!ok) break;
                const int ts0 = t0 + s * SLAB;
                const bool zero_halo = (ts0 == 0) && (f.cs_in == nullptr);
                const int nvalid = min(SLAB, T - ts0) - tg * 16;  // tokens of this thread's group that exist
                const uint8_t *xs = smem + SMEM_X + slot * X_SLAB_BYTES + x_thread_off + (uint32_t)(tg * 16) * X_ROW_BYTES;
                auto load_row = [&](int r, f32x2 &v01, f32x2 &v23) {   // r: row relative to this thread's first halo row
                    const uint2 w = *(const uint2 *)(xs + (uint32_t)r * X_ROW_BYTES);
                    v01 = pack2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u));
                    v23 = pack2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
                };
                // row of token i of this thread: rowbase + 2 i; its 16-byte chunk is swizzled by (row & 7) = (p + 2 i) & 7
                const uint32_t pbit = (uint32_t)(s & 1);
                const uint32_t row_addr = u_base + (uint32_t)((s >> 1) * 64 + (s & 1) + 32 * tg) * 128u;
                uint32_t sw[4];
#pragma unroll
                for (int m = 0; m < 4; ++m) sw[m] = row_addr + ((u_chunk ^ ((pbit + 2u * m) & 7u)) << 4);
                if (nvalid > 0) {
                    f32x2 a01, a23, b01x, b23x, c01, c23;  // x_{t-3}, x_{t-2}, x_{t-1}
                    load_row(0, a01, a23); load_row(1, b01x, b23x); load_row(2, c01, c23);
                    if (zero_halo && tg == 0) { a01 = a23 = b01x = b23x = c01 = c23 = pack2(0.f, 0.f); }
                    if (nvalid >= 16) {
                        // four tokens at a time, tap by tap, so that eight independent FMA chains are in flight
                        f32x2 h01[3] = {a01, b01x, c01}, h23[3] = {a23, b23x, c23};
#pragma unroll
                        for (int i0 = 0; i0 < 16; i0 += 4) {
                            f32x2 r01[7], r23[7];   // rows t-3 .. t+3 of the batch
#pragma unroll
                            for (int k = 0; k < 3; ++k) { r01[k] = h01[k]; r23[k] = h23[k]; }
#pragma unroll
                            for (int k = 0; k < 4; ++k) load_row(3 + i0 + k, r01[3 + k], r23[3 + k]);
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
                                *(uint2 *)(smem + sw[(i0 + k) & 3] + (uint32_t)(i0 + k) * 256u) =
                                    make_uint2(pack_f16_sat(lo2(u01[k]), hi2(u01[k])), pack_f16_sat(lo2(u23[k]), hi2(u23[k])));
#pragma unroll
                            for (int k = 0; k < 3; ++k) { h01[k] = r01[4 + k]; h23[k] = r23[4 + k]; }
                        }
                    } else {
                        for (int i = 0; i < nvalid; ++i) {
                            f32x2 d01, d23;
                            load_row(3 + i, d01, d23);
                            f32x2 u01 = fma2(w01[0], d01, b01), u23 = fma2(w23[0], d23, b23);
                            u01 = fma2(w01[1], c01, u01); u23 = fma2(w23[1], c23, u23);
                            u01 = fma2(w01[2], b01x, u01); u23 = fma2(w23[2], b23x, u23);
                            u01 = fma2(w01[3], a01, u01); u23 = fma2(w23[3], a23, u23);
                            const uint32_t addr = row_addr + ((u_chunk ^ ((pbit + 2u * (uint32_t)i) & 7u)) << 4) + (uint32_t)i * 256u;
                            *(uint2 *)(smem + addr) = make_uint2(pack_f16_sat(lo2(u01), hi2(u01)), pack_f16_sat(lo2(u23), hi2(u23)));
                            a01 = b01x; a23 = b23x; b01x = c01; b23x = c23; c01 = d01; c23 = d23;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(BAR_XEMPTY(slot));
            }
            if (!ok) break;
            fence_async_smem();  // make the generic-proxy writes of U visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR_UFULL(st));
        }
        if (!ok && lane == 0) record_timeout(f.status, abort_flag);
    } else if (warp < 8) {
      reg_dec<40>();
      if (warp == 4) {
        // ================================================================ TMA loader
        const __nv_bfloat16 *x = (const __nv_bfloat16 *)f.x;
        const __nv_bfloat16 *cs_in = (const __nv_bfloat16 *)f.cs_in;
        int slab_n = 0;
        bool ok = true;
        int b, ti;
        tile_first(b, ti);
        for (int it = 0; it < n_my_tiles && ok; tile_next(it, b, ti), ++it) {
            const int t0 = ti * TILE_N;
            const int nslab = min(TILE_N / SLAB, (T - t0 + SLAB - 1) / SLAB);
            for (int s = 0; s < nslab; ++s, ++slab_n) {
                const int slot = slab_n % XS;
                ok = warp_wait(BAR_XEMPTY(slot), ((slab_n / XS) & 1) ^ 1, spin, abort_flag);
                if (!ok) break;
                const int ts0 = t0 + s * SLAB;
                const uint32_t dst = base + SMEM_X + slot * X_SLAB_BYTES;
                if (ts0 == 0 && cs_in != nullptr) {
                    // first slab of a sequence with an incoming conv state: the three halo rows come from
                    // conv_state_in, so the slab is assembled from row copies
                    const int hi_row = min(SLAB_ROWS, T + 3);
                    if (lane == 0) mbar_expect_tx(BAR_XFULL(slot), (uint32_t)hi_row * X_ROW_BYTES);
                    __syncwarp();
                    for (int r = lane; r < hi_row; r += 32) {
                        const int t = r - 3;
                        const __nv_bfloat16 *src = t >= 0 ? x + ((size_t)b * T + t) * D + head * DH
                                                          : cs_in + ((size_t)b * 3 + (3 + t)) * D + head * DH;
                        bulk_g2s(dst + r * X_ROW_BYTES, src, X_ROW_BYTES, BAR_XFULL(slot));
                    }
                } else if (lane == 0) {
                    // one tiled copy per slab: SLAB_ROWS token rows of this head starting three tokens early
                    // (tokens before the sequence start and past its end read as zero)
                    mbar_expect_tx(BAR_XFULL(slot), X_SLAB_BYTES);
                    tma_load_3d(dst, &p.tm_x, head * DH, ts0 - 3, b, BAR_XFULL(slot));
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) record_timeout(f.status, abort_flag);
      } else if (warp == 5 || warp == 6) {
        // ================================================================ MMA issuers: warp 5 the W_a products, warp 6 the W_x products
        // (one thread's issue stream runs at 70-85 cycles per instruction beside the busy warps of its scheduler;
        // two streams on two schedulers keep the tensor pipe fed)
        const uint32_t tm_w = warp == 5 ? TM_W_A : TM_W_X, tm_acc = warp == 5 ? TM_ACC_A : TM_ACC_X;
        // One N = 128 instruction per gate and K step: an N = 64 instruction takes about 45 cycles where 32 would be
        // its share, an N = 128 one the full-rate 64, so halves would cost more tensor time than they overlap.
        constexpr uint32_t idesc = make_idesc_f16(128, TILE_N);
        bool ok = true;
        if (lane == 0) {
            ok = mbar_wait(BAR_WREADY, 0, spin, abort_flag);
            for (int it = 0; it < n_my_tiles && ok; ++it) {
                const int st = it % US;
                ok = mbar_wait(BAR_UFULL(st), (it / US) & 1, spin, abort_flag);
                if (!ok) break;
                const uint32_t u_base = base + SMEM_U + st * U_STAGE_BYTES;
                ok = mbar_wait(BAR_ACCEMPTY(0), (it & 1) ^ 1, spin, abort_flag);
                if (!ok) break;
                tc_fence_after();
                // the start-address field of the descriptor counts 16-byte units
                const uint64_t bd0 = make_desc_sw128(u_base);
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    const uint64_t bd = bd0 + (uint64_t)(((ks >> 2) * U_KBLOCK_BYTES + (ks & 3) * 32) >> 4);
                    mma_ts(tmem + tm_acc, tmem + tm_w + ks * 8, bd, idesc, ks > 0);
                }
                tc_commit(BAR_UEMPTY(st));
                tc_commit(BAR_ACCFULL(0));
            }
            if (!ok) record_timeout(f.status, abort_flag);
        }
        __syncwarp();
      }
    } else {
        // ================================================================ epilogue
        reg_inc<200>();
        const int q = warp & 3, k = (warp - 8) >> 2;
        const int c_own = q * 32 + lane;                 // channel within the CTA
        const int hc = half * CH + c_own;                // channel within the head
        const int d = head * DH + hc;                    // global channel
        // per-channel constants; s = c softplus(-Lambda) with libm-grade log1p/exp (Appendix A)
        const float lam = f.lambda[d];
        const float zl = -lam;
        const float s = f.c * (zl > 0.0f ? zl + log1pf(expf(-zl)) : log1pf(expf(zl)));
        const f32x2 s2 = pack2(s, s);
        const f32x2 hba2 = pack2(0.5f * f.b_a[d], 0.5f * f.b_a[d]), hbx2 = pack2(0.5f * f.b_x[d], 0.5f * f.b_x[d]);
        const bool poly = __all_sync(0xffffffffu, s <= S_POLY);
        // u[row][channel] in the swizzled U tile, one offset per row phase (row & 7)
        uint32_t u_off[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            u_off[j] = (uint32_t)(hc >> 6) * U_KBLOCK_BYTES + ((((uint32_t)(hc & 63) >> 3) ^ (uint32_t)j) << 4) + (uint32_t)(hc & 7) * 2 +
                       (uint32_t)(k * EPI_TOK) * 128u;
        const uint32_t tm_lane = tmem + ((uint32_t)(q * 32) << 16);
        const uint32_t y_warp_off = SMEM_Y + (uint32_t)(k * 4 + q) * Y_WARP_BYTES;
        uint16_t *y_s = (uint16_t *)(smem + y_warp_off) + lane;   // this thread's column of the warp's y block [64 tokens][32 channels]
        const uint32_t y_s_addr = base + y_warp_off;
        const __nv_bfloat16 *x = (const __nv_bfloat16 *)f.x;
        const __nv_bfloat16 *cs_in = (const __nv_bfloat16 *)f.cs_in;
        float h_prev_own = 0.0f;  // state at the end of this CTA's previous tile
        float h_scan_end = 0.0f;  // state at the end of this warp's 64 tokens of the previous tile
        bool ok = true;
        int b, ti;
        tile_first(b, ti);
        for (int it = 0; it < n_my_tiles && ok; tile_next(it, b, ti), ++it) {
            const bool shared = it < n_shared;
            const int g = b * p.tps + ti;   // tile number within the half-head: index of its carry record
            const int t0 = ti * TILE_N;
            const int st = it % US;
            const int nv = max(0, min(EPI_TOK, T - t0 - k * EPI_TOK));  // valid tokens of this warp
            if (k == 0 && it > 0) {
                // The first half left the previous tile without the second half's fold; it takes it now, before its own
                // next arrival on BAR_AGG (so that neither side is ever more than one barrier phase ahead of the other).
                ok = warp_wait(BAR_AGG(q, 1), (it - 1) & 1, spin, abort_flag);
                if (!ok) break;
                const float2 other = agg_s[((((it - 1) & 1) * 2 + 1) * 4 + q) * 32 + lane];
                h_prev_own = fmaf(other.x, h_scan_end, other.y);
            }
            ok = warp_wait(BAR_ACCFULL(0), it & 1, spin, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // A2[j] / V2[j]: tokens j (low half) and j + 32 (high half) of this warp's 64 tokens
            f32x2 A2[EPI_TOK / 2], V2[EPI_TOK / 2];
            tmem_ld32(tm_lane + TM_ACC_A + k * EPI_TOK, A2);
            tmem_ld32(tm_lane + TM_ACC_A + k * EPI_TOK + 32, A2 + 16);
            tmem_ld32(tm_lane + TM_ACC_X + k * EPI_TOK, V2);
            tmem_ld32(tm_lane + TM_ACC_X + k * EPI_TOK + 32, V2 + 16);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR_ACCEMPTY(0));  // the accumulators now live in registers
            // gates, decay, input scale: (z_a, z_x) -> (a_t, v_t) in place
            const uint8_t *u_tile = smem + SMEM_U + st * U_STAGE_BYTES;
            auto gates = [&](auto poly_tag) {
                constexpr bool POLY = decltype(poly_tag)::value;
#pragma unroll
                for (int j = 0; j < EPI_TOK / 2; j += 4) {
                    float u[8];   // rows 2j' (token j') and 2j' + 1 (token j' + 32) for j' = j .. j + 3
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        u[e] = f16_bits_to_f32(*(const uint16_t *)(u_tile + u_off[(2 * j + e) & 7] + (uint32_t)(2 * j + e) * 128u));
                    gate_group<POLY, 4>(A2 + j, V2 + j, u, hba2, hbx2, s2);
                }
            };
            if (poly) gates(std::true_type{}); else gates(std::false_type{});
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR_UEMPTY(st));  // done reading u
            if (nv < EPI_TOK) {
                // ragged tail: tokens that do not exist hold the state (a = 1, v = 0)
#pragma unroll
                for (int j = 0; j < EPI_TOK / 2; ++j) {
                    const bool v0 = j < nv, v1 = j + 32 < nv;
                    A2[j] = pack2(v0 ? lo2(A2[j]) : 1.0f, v1 ? hi2(A2[j]) : 1.0f);
                    V2[j] = pack2(v0 ? lo2(V2[j]) : 0.0f, v1 ? hi2(V2[j]) : 0.0f);
                }
            }
            // ---- fold both halves at once: h_out = P h_in + hl for tokens [0,32) (low) and [32,64) (high)
            f32x2 P2 = pack2(1.0f, 1.0f), HL2 = pack2(0.0f, 0.0f);
#pragma unroll
            for (int j = 0; j < EPI_TOK / 2; ++j) { P2 = mul2(P2, A2[j]); HL2 = fma2(A2[j], HL2, V2[j]); }
            const float P_lo = lo2(P2), hl_lo = lo2(HL2);
            const float P = P_lo * hi2(P2), hl = fmaf(hi2(P2), hl_lo, hi2(HL2));
            // ---- the second half of the tile needs the fold of the first; the first half goes on without waiting
            //      and picks up the second half's fold at the start of the next tile
            //      (the second half arrives only after its own wait: then neither barrier can run two phases ahead)
            agg_s[(((it & 1) * 2 + k) * 4 + q) * 32 + lane] = make_float2(P, hl);
            float P_0 = P, hl_0 = hl, P_t = 0.0f, hl_t = 0.0f;    // tokens [0, 64); whole tile (second half only)
            if (k == 1) {
                ok = warp_wait(BAR_AGG(q, 0), it & 1, spin, abort_flag);
                if (!ok) break;
                const float2 other = agg_s[(((it & 1) * 2 + 0) * 4 + q) * 32 + lane];
                P_0 = other.x; hl_0 = other.y;
                P_t = P_0 * P; hl_t = fmaf(P, hl_0, hl);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR_AGG(q, k));
            if (shared && S > 1 && k == 1) {
                uint4 rec;
                rec.x = __float_as_uint(P_t); rec.y = p.tag; rec.z = __float_as_uint(hl_t); rec.w = p.tag;
                uint4 *dst = p.agg + ((size_t)group * p.tiles_total + g) * CH + c_own;
                asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(rec.x), "r"(rec.y), "r"(rec.z), "r"(rec.w) : "memory");
            }
            // ---- incoming state of the tile (both halves work it out for themselves): the state this CTA
            //      reached at the end of its previous tile, or h0 near the start of a sequence, advanced by
            //      the aggregates that the other CTAs published for the tiles in between (decoupled look-back)
            float h;
            int nback;
            if (!shared) {
                h = ti == 0 ? (f.h0 ? f.h0[(size_t)b * D + d] : 0.0f) : h_prev_own;
                nback = 0;
            } else if (ti == 0 || (S > 1 && ti < S)) {
                h = f.h0 ? f.h0[(size_t)b * D + d] : 0.0f;
                nback = ti;
            } else {
                h = h_prev_own;
                nback = S - 1;
            }
            if (nback > 0) {
                // All records are requested at once, then polled until every lane sees this call's tag in
                // both halves of each record (8-byte words are written atomically).
                const uint4 *src = p.agg + ((size_t)group * p.tiles_total + g) * CH + c_own;
                uint4 rec[MAX_S - 1];
                uint64_t tstart = 0;
                for (uint32_t npoll = 0;; ++npoll) {
                    bool ready = true;
#pragma unroll
                    for (int j = 1; j < MAX_S; ++j) {
                        if (j <= nback) {
                            const uint4 *sj = src - (size_t)j * CH;
                            asm volatile("ld.volatile.global.v4.b32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(rec[j - 1].x), "=r"(rec[j - 1].y), "=r"(rec[j - 1].z), "=r"(rec[j - 1].w) : "l"(sj) : "memory");
                        }
                    }
#pragma unroll
                    for (int j = 1; j < MAX_S; ++j)
                        if (j <= nback) ready = ready && rec[j - 1].y == p.tag && rec[j - 1].w == p.tag;
                    if (__all_sync(0xffffffffu, ready)) break;
                    if ((npoll & 15u) == 15u) {
                        const uint64_t tnow = gtimer();
                        if (tstart == 0) tstart = tnow;
                        if (*abort_flag || tnow - tstart > spin) { ok = false; break; }
                    }
                    __nanosleep(32);
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
#pragma unroll
                for (int j = MAX_S - 1; j >= 1; --j)
                    if (j <= nback) h = fmaf(__uint_as_float(rec[j - 1].x), h, __uint_as_float(rec[j - 1].z));
            }
            if (k == 1) h_prev_own = fmaf(P_t, h, hl_t);   // state at the end of this tile (the first half works it out later)
            if (k == 1) h = fmaf(P_0, h, hl_0);       // state at the start of the second half
            // ---- the warp's y block must have been read out by its previous tiled store
            if (lane == 0) bulk_wait_read0();
            __syncwarp();
            // ---- the recurrence h_t = a_t h_{t-1} + v_t (Eq. 4), both halves in lock step; y_t = h_t
            f32x2 H2 = pack2(h, fmaf(P_lo, h, hl_lo));
#pragma unroll
            for (int j = 0; j < EPI_TOK / 2; ++j) {
                H2 = fma2(A2[j], H2, V2[j]);
                const __nv_bfloat162 o = __floats2bfloat162_rn(lo2(H2), hi2(H2));
                const uint32_t ow = *(const uint32_t *)&o;
                y_s[j * 32] = (uint16_t)(ow & 0xFFFFu);             // row j of the warp's block: 32 channels x 2 bytes
                y_s[(j + 32) * 32] = (uint16_t)(ow >> 16);
            }
            h = hi2(H2);
            h_scan_end = h;
            fence_async_smem();   // y rows become visible to the bulk-copy engine
            __syncwarp();
            if (lane == 0) {
                // the warp's 64 tokens x 32 channels go out as one tiled store; rows at or beyond T are clipped
                if (nv > 0) tma_store_3d(&p.tm_y, head * DH + half * CH + q * 32, t0 + k * EPI_TOK, b, y_s_addr);
                bulk_commit();
            }
            if (k == 1 && ti == p.tps - 1) {
                // end of a sequence: h_T (unrounded state) and the last three raw inputs, bit-exact
                f.h_T[(size_t)b * D + d] = h;
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
        if (!ok && lane == 0) record_timeout(f.status, abort_flag);
    }

    // ---- teardown: every role falls through to here, also after a timeout
    if (*abort_flag) {
        // let copies and MMAs in flight land before shared and tensor memory are given back
        const uint64_t tw = gtimer();
        while (gtimer() - tw < 50000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tmem, 512);
}

int num_sms() {
    static int cached = 0;
    if (cached == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached = n;
        else
            return 148;
    }
    return cached;
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

bool sm100_prefill_supported(int B, int T, int D, int H, int io) {
    return io == RGLRU_BF16 && B > 0 && T > 0 && H > 0 && D == H * DH;
}

namespace {
inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }
size_t agg_bytes(int B, int T, int H) {
    const size_t tps = (T + TILE_N - 1) / TILE_N;
    return up256((size_t)H * 2 * B * tps * CH * sizeof(uint4));
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
    return agg_bytes(B, T, H) + up256((size_t)B * D * sizeof(float)) + up256((size_t)B * 3 * D * sizeof(__nv_bfloat16));
}

cudaError_t sm100_prefill(const FwdArgs &a, void *ws_body, size_t ws_body_bytes, cudaStream_t st) {
    static bool attr_set = false;
    cudaError_t e;
    if (!attr_set) {
        e = cudaFuncSetAttribute(sm100_prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    Sm100Args p;
    if (!make_activation_map(&p.tm_x, a.x, a.B, a.T, a.D, DH, SLAB_ROWS) || !make_activation_map(&p.tm_y, a.y, a.B, a.T, a.D, 32, EPI_TOK))
        return cudaErrorNotSupported;
    p.f = a;
    p.tps = (a.T + TILE_N - 1) / TILE_N;
    p.tiles_total = a.B * p.tps;
    const int groups = a.H * 2;
    const int nsm = num_sms();
    int S = nsm / groups;
    if (S < 1) S = 1;
    if (S > MAX_S) S = MAX_S;
    if (S > p.tiles_total) S = p.tiles_total;
    p.S = S;
    p.tag = next_tag();
    p.agg = (uint4 *)ws_body;
    p.spin_ns = g_spin_limit_ns;
    if (ws_body_bytes < sm100_prefill_workspace_bytes(a.B, a.T, a.D, a.H)) return cudaErrorInvalidValue;
    const size_t h_bytes = (size_t)a.B * a.D * sizeof(float), cs_bytes = (size_t)a.B * 3 * a.D * sizeof(__nv_bfloat16);
    char *h0_copy = (char *)ws_body + agg_bytes(a.B, a.T, a.H), *cs_copy = h0_copy + up256(h_bytes);
    if (ranges_overlap(a.h0, a.h_T, h_bytes)) {
        if ((e = cudaMemcpyAsync(h0_copy, a.h0, h_bytes, cudaMemcpyDeviceToDevice, st)) != cudaSuccess) return e;
        p.f.h0 = (const float *)h0_copy;
    }
    if (ranges_overlap(a.cs_in, a.cs_out, cs_bytes)) {
        if ((e = cudaMemcpyAsync(cs_copy, a.cs_in, cs_bytes, cudaMemcpyDeviceToDevice, st)) != cudaSuccess) return e;
        p.f.cs_in = cs_copy;
    }
    dim3 grid(groups * S), block(NUM_THREADS);
    if (S > 1) {
        // CTAs wait on one another's aggregates: they must all be resident
        void *args[] = {(void *)&p};
        return cudaLaunchCooperativeKernel((const void *)sm100_prefill_kernel, grid, block, args, SMEM_ALLOC, st);
    }
    sm100_prefill_kernel<<<grid, block, SMEM_ALLOC, st>>>(p);
    return cudaGetLastError();
}

}  // namespace rglru
