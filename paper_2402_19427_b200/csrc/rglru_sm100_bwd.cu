// sm_100a backward of the RG-LRU temporal core (bf16 io, head width a multiple of 32 up to 256 -- narrower heads in groups of
// 256 channel slots --, T a multiple of 8).
//
// The paper gives no backward; this is reverse-mode differentiation of Eq. 1-4 and the Conv1D.  The three dense
// contractions run on tcgen05 tensor cores through one small GEMM kernel, the rest is element-wise and HBM-bound:
//   1. conv_forward      u = Conv1D(x) in fp16, token-major [tok][D]; fp16 copies of the weights
//                        (every tensor-core operand here is fp16: 11 significant bits instead of bf16's 8 keep the
//                        rounding of u and dz out of the gradients; finite overflow saturates at +-65504)
//   2. GEMM              z_a | z_x = u W_a^T | u W_x^T per head (Eq. 1-2 before the sigmoid), fp16 out
//   3. scan_fold / scan_carry / scan_apply
//                        reverse-time scan g_t = dy_t + a_{t+1} g_{t+1} over chunks of 128 tokens (fold, carry across
//                        chunks, re-run with the carry), then the element-wise adjoints: dz_a, dz_x (fp16, token-major),
//                        the direct part of du (fp16), partial sums of dLambda, db_a, db_x
//   4. GEMM              du += dz_a W_a + dz_x W_x
//   5. GEMM (split K)    dW_a | dW_x = dz^T u over all tokens: both operands are read token-major as steps 1 and 3 wrote them
//                        and handed to the tensor core as MN-major operands (no transposed copies exist); fp32 partial sums
//                        per split, reduced in fixed order
//   6. Conv1D adjoint    dx, dconv_w, dconv_b with sliding windows, fixed-order reductions
// h_{t-1} comes from the forward output y (bf16); when the caller has none the forward is run first.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "rglru_internal.h"
#include "sm100_ptx.cuh"

namespace rglru {
namespace {

using namespace ptx;

constexpr int DH = 256;
constexpr int CHUNK = 128;                 // tokens per scan chunk = rows of a GEMM tile
constexpr int GEMM_THREADS = 192;          // TMA warp, MMA warp, four epilogue warps
constexpr int GEMM_STAGES = 4;
constexpr uint32_t A_STAGE_BYTES = 128 * 128;   // 128 rows x 64 bf16
constexpr uint32_t B_STAGE_BYTES = 256 * 128;   // 256 rows x 64 bf16
constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr uint32_t MN_BLOCK_BYTES = 64 * 128;   // one copy of 64 tokens x 64 channels for the MN-major operands of the dW product
constexpr uint32_t GEMM_SMEM_BAR = GEMM_STAGES * STAGE_BYTES;
constexpr uint32_t GEMM_SMEM_TOTAL = GEMM_SMEM_BAR + (2 * GEMM_STAGES + 4) * 8 + 16;
constexpr uint32_t GEMM_SMEM_ALLOC = GEMM_SMEM_TOTAL + 1024;

enum { MODE_Z = 0, MODE_DU = 1, MODE_DW = 2 };

struct GemmArgs {
    alignas(64) CUtensorMap tm_a;    // A rows (M side), K innermost
    alignas(64) CUtensorMap tm_b0;   // B rows (N side), K innermost
    alignas(64) CUtensorMap tm_b1;   // MODE_Z: the second gate's weights (grid.y selects)
    int mode, H, D;    // H: 256-slot groups of heads
    int hstride;       // channels from one group to the next in the layer's [.., D] arrays (k dh with k = 256 / dh heads per group)
    int cvalid;        // channel slots of a group that exist (k dh; fewer in a partial last group)
    int nx, ny;        // tile grid: nx x ny x H
    int kblocks;       // 64-wide K blocks per CTA
    int rows_valid;    // MODE_Z / MODE_DU: number of tokens; MODE_DW: 512
    void *out;         // MODE_Z: __half z[tok][H][2][256]; MODE_DU: __half du[tok][D] (+=); MODE_DW: float part[split][2][H][256][256]
    uint32_t *status;
    unsigned long long spin_ns;
};

// C[128 x 256] = A[128 x K] B[256 x K]^T per tile; A and B tiles arrive by tiled TMA in the 128-byte-swizzled K-major
// layout, accumulate in tensor memory (fp32), and leave through the four epilogue warps.  CTAs are persistent: each
// walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... with two accumulators, so that the epilogue of one tile overlaps
// the loads and MMAs of the next.  Tile number -> (x, y, z) with x fastest:
//   MODE_Z : (token tiles, 2 gates, H)   A = u[tok][h][k]        B = W_gate[h][out][k]
//   MODE_DU: (token tiles, 1, H)         A = dz[tok][h][k=512]   B = W^T[h][in][k=512]
//   MODE_DW: (4 row tiles, splits, H)    A = dz[tok][h][row]     B = u[tok][h][in], both MN-major, K = this split's tokens
// 32-byte accesses: one whole DRAM sector per thread and instruction where a thread owns a row (pointers 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void *ptr, const uint32_t (&r)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(ptr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]),
                 "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void ld_global_v8(const void *ptr, uint32_t (&r)[8]) {
    asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]),
                 "=r"(r[6]), "=r"(r[7]) : "l"(ptr) : "memory");
}

__global__ void __launch_bounds__(GEMM_THREADS, 1) tc_gemm_kernel(const __grid_constant__ GemmArgs p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    const uint32_t bar0 = base + GEMM_SMEM_BAR;
    auto BAR_FULL = [&](int s) { return bar0 + 8u * s; };
    auto BAR_EMPTY = [&](int s) { return bar0 + 8u * (GEMM_STAGES + s); };
    auto BAR_ACCFULL = [&](int a) { return bar0 + 8u * (2 * GEMM_STAGES + a); };
    auto BAR_ACCEMPTY = [&](int a) { return bar0 + 8u * (2 * GEMM_STAGES + 2 + a); };
    uint32_t *tmem_base_s = (uint32_t *)(smem + GEMM_SMEM_BAR + (2 * GEMM_STAGES + 4) * 8);
    volatile int *abort_flag = (volatile int *)(tmem_base_s + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const unsigned long long spin = p.spin_ns;
    const int ntiles = p.nx * p.ny * p.H;
    // Tiles are dealt round-robin.  (Contiguous runs per CTA, with the B operand left in shared memory while head and gate
    // stay the same, measured 4 % slower on the whole backward: the operand re-reads hit L2 and were not the limit.)

    if (tid == 0) {
        for (int s = 0; s < GEMM_STAGES; ++s) { mbar_init(BAR_FULL(s), 1); mbar_init(BAR_EMPTY(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(BAR_ACCFULL(a), 1); mbar_init(BAR_ACCEMPTY(a), 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) { tmem_alloc(smem_u32(tmem_base_s), 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_base_s;
    bool ok = true;

    if (warp == 0) {
        // ---- TMA producer
        if (lane == 0) {
            int kbg = 0;   // K blocks issued so far, over all tiles (ring position)
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int tx = tile % p.nx, ty = (tile / p.nx) % p.ny, h = tile / (p.nx * p.ny);
                const CUtensorMap *tb = (p.mode == MODE_Z && ty == 1) ? &p.tm_b1 : &p.tm_b0;
                for (int kb = 0; kb < p.kblocks; ++kb, ++kbg) {
                    const int s = kbg % GEMM_STAGES;
                    ok = mbar_wait(BAR_EMPTY(s), ((kbg / GEMM_STAGES) & 1) ^ 1, spin, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(BAR_FULL(s), STAGE_BYTES);
                    const uint32_t a_dst = base + s * STAGE_BYTES, b_dst = a_dst + A_STAGE_BYTES;
                    if (p.mode == MODE_DW) {
                        // both operands token-major as the scan wrote them: 64 tokens (K) x 64 channels per copy, the channels
                        // innermost; tokens at or beyond B T read as zero
                        const int k0 = (ty * p.kblocks + kb) * 64;
#pragma unroll
                        for (int j = 0; j < 2; ++j) tma_load_3d(a_dst + j * MN_BLOCK_BYTES, &p.tm_a, tx * 128 + j * 64, h, k0, BAR_FULL(s));
#pragma unroll
                        for (int j = 0; j < 4; ++j) tma_load_3d(b_dst + j * MN_BLOCK_BYTES, tb, h * p.hstride + j * 64, k0, 0, BAR_FULL(s));
                    } else {
                        // u is read out of the layer's [tok][D] array at the group's first channel (channels past the group's own
                        // meet zero weights; past D they read as zero); dz has the groups' own [tok][group][2][256] layout
                        if (p.mode == MODE_Z) tma_load_3d(a_dst, &p.tm_a, h * p.hstride + kb * 64, tx * 128, 0, BAR_FULL(s));
                        else tma_load_3d(a_dst, &p.tm_a, kb * 64, h, tx * 128, BAR_FULL(s));
                        tma_load_3d(b_dst, tb, kb * 64, 0, h, BAR_FULL(s));
                    }
                }
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT); }
        }
    } else if (warp == 1) {
        // ---- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_f16(128, 256), idesc_mn = make_idesc_f16_mn(128, 256);
            int kbg = 0, it = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++it) {
                const int acc = it & 1;
                ok = mbar_wait(BAR_ACCEMPTY(acc), ((it >> 1) & 1) ^ 1, spin, abort_flag);   // epilogue of tile it - 2 done
                if (!ok) break;
                for (int kb = 0; kb < p.kblocks; ++kb, ++kbg) {
                    const int s = kbg % GEMM_STAGES;
                    ok = mbar_wait(BAR_FULL(s), (kbg / GEMM_STAGES) & 1, spin, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_src = base + s * STAGE_BYTES, b_src = a_src + A_STAGE_BYTES;
                    if (p.mode == MODE_DW) {
                        // K = tokens runs along the rows of the staged blocks: 16 rows of 128 bytes per instruction
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_ss(tmem + acc * 256, make_desc_sw128_mn(a_src + ks * 2048, MN_BLOCK_BYTES), make_desc_sw128_mn(b_src + ks * 2048, MN_BLOCK_BYTES),
                                   idesc_mn, (kb | ks) != 0);
                    } else {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_ss(tmem + acc * 256, make_desc_sw128(a_src + ks * 32), make_desc_sw128(b_src + ks * 32), idesc, (kb | ks) != 0);
                    }
                    tc_commit(BAR_EMPTY(s));
                }
                if (ok) tc_commit(BAR_ACCFULL(acc));
            }
            if (!ok) { *abort_flag = 1; atomicExch(p.status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT); }
        }
    } else {
        // ---- epilogue: warp owns TMEM lanes 32 (warp & 3) .. +31 = rows of the tile
        const int q = warp & 3;
        int it = 0;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++it) {
            const int tx = tile % p.nx, ty = (tile / p.nx) % p.ny, h = tile / (p.nx * p.ny);
            const int acc = it & 1;
            const int row = tx * 128 + q * 32 + lane;
            ok = warp_wait(BAR_ACCFULL(acc), (it >> 1) & 1, spin, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t tm_lane = tmem + ((uint32_t)(q * 32) << 16) + acc * 256;
            const bool valid = row < p.rows_valid;
            const int cv = min(p.cvalid, p.D - h * p.hstride);   // channel slots of this group that exist
#pragma unroll 1
            for (int c0 = 0; c0 < 256; c0 += 32) {
                f32x2 v[16];
                tmem_ld32(tm_lane + c0, v);
                tmem_ld_wait();
                if (!valid) continue;
                if (p.mode == MODE_Z) {
                    __half *dst = (__half *)p.out + (((size_t)row * p.H + h) * 2 + ty) * 256 + c0;
#pragma unroll
                    for (int j8 = 0; j8 < 2; ++j8) {
                        uint32_t w[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) { const __half2 hh = __floats2half2_rn(lo2(v[8 * j8 + j]), hi2(v[8 * j8 + j])); w[j] = *(const uint32_t *)&hh; }
                        st_global_v8(dst + 16 * j8, w);
                    }
                } else if (p.mode == MODE_DU) {
                    // du is kept in fp16 like dz (bf16 failed the dx tolerance where the taps of the Conv1D adjoint cancel)
                    if (c0 >= cv) continue;   // a slot that does not exist: nothing of du belongs to it
                    __half *dst = (__half *)p.out + (size_t)row * p.D + h * p.hstride + c0;
                    uint32_t o0[8], o1[8];
                    ld_global_v8(dst, o0);
                    ld_global_v8(dst + 16, o1);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float2 a0 = __half22float2(*(const __half2 *)&o0[j]), a1 = __half22float2(*(const __half2 *)&o1[j]);
                        o0[j] = pack_f16_sat(a0.x + lo2(v[j]), a0.y + hi2(v[j]));
                        o1[j] = pack_f16_sat(a1.x + lo2(v[8 + j]), a1.y + hi2(v[8 + j]));
                    }
                    st_global_v8(dst, o0);
                    st_global_v8(dst + 16, o1);
                } else {
                    const int g = row >> 8, o_row = row & 255;
                    float *dst = (float *)p.out + ((((size_t)ty * 2 + g) * p.H + h) * 256 + o_row) * 256 + c0;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t w[8];
#pragma unroll
                        for (int e = 0; e < 4; ++e) { w[2 * e] = __float_as_uint(lo2(v[4 * j + e])); w[2 * e + 1] = __float_as_uint(hi2(v[4 * j + e])); }
                        st_global_v8(dst + 8 * j, w);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR_ACCEMPTY(acc));   // this accumulator may be overwritten
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicExch(p.status, STATUS_MAGIC | (uint32_t)RGLRU_ERR_TIMEOUT); }
    }
    if (*abort_flag) {   // let copies and MMAs in flight land before shared and tensor memory are given back
        const uint64_t tw = gtimer();
        while (gtimer() - tw < 50000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------ element-wise kernels
__device__ __forceinline__ float bf2f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float sigmoid_acc(float z) { return 1.0f / (1.0f + expf(-z)); }
// Hardware-approximate versions for the per-element work (relative error ~1e-6, far inside the gradient tolerance)
__device__ __forceinline__ float rcp_fast(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float rsqrt_fast(float x) { float y; asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float sigmoid_fast(float z) { return rcp_fast(1.0f + __expf(-z)); }
// 1 - exp(x) for x <= 0 without cancellation near 0
__device__ __forceinline__ float one_minus_exp(float x) {
    if (x > -0.25f) {   // -x (1 + x/2 + x^2/6 + x^3/24 + x^4/120 + x^5/720): relative truncation error < 2e-7
        float pl = fmaf(x, 1.0f / 720.0f, 1.0f / 120.0f);
        pl = fmaf(pl, x, 1.0f / 24.0f); pl = fmaf(pl, x, 1.0f / 6.0f); pl = fmaf(pl, x, 0.5f); pl = fmaf(pl, x, 1.0f);
        return -x * pl;
    }
    return 1.0f - __expf(x);
}
// s = c softplus(-Lambda)   (Appendix A, with a = sigmoid(Lambda))
__device__ __forceinline__ float decay_rate(float lambda, float c) {
    const float z = -lambda;
    return c * (z > 0.0f ? z + log1pf(expf(-z)) : log1pf(expf(z)));
}

struct EwArgs {
    int B, T, D, H, nchunk;
    int hstride;                      // channels from one 256-slot group of heads to the next
    float c;
    const __nv_bfloat16 *x, *conv_w, *cs_in, *dy, *y;
    const float *conv_b, *b_a, *b_x, *lambda, *h0;
    __half *u, *dz;
    const __half *z;
    __half *du;                       // [tok][D]
    float2 *fold;                     // [B][nchunk][D]: (prod a_t, carry out of the chunk for zero carry in)
    float *xin;                       // [B][nchunk][D]: a_{t+1} g_{t+1} entering the chunk from later tokens
    float *part_vec;                  // [B*nchunk][3][D]
    const float *dh_T;                // [B][D] gradient arriving on h_T, or null
    float *dh0;                       // [B][D] gradient of h0, or null
};

// fp16 copies of the gate weights: W16[g][h][o][n] = W_g[h][o][n] and WT[h][n][g*256 + o] = W_g[h][o][n]
// One block per 32 x 32 tile of one (gate, head) matrix; the transposed copy goes through shared memory so that both
// copies are written with consecutive threads on consecutive addresses.  grid (8, 8, 2 H), block (32, 8)
// H counts 256-slot groups; dh is the width of a head of the layer (a multiple of 32 up to 256): a group holds k = 256 / dh
// (rounded down) heads on its diagonal -- fewer in a partial last group of a layer of Hl heads -- and every tile outside
// those blocks is written as zeros.
__global__ void convert_w_kernel(const __nv_bfloat16 *Wa, const __nv_bfloat16 *Wx, __half *W16, __half *WT, int H, int dh, int Hl) {
    __shared__ __half tile[32][33];
    const int g = blockIdx.z / H, h = blockIdx.z % H;
    const int o0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
    const int k = DH / dh, sub = o0 / dh;            // heads per group; head of the group that owns these output rows
    const int heads_here = min(k, Hl - h * k);
    const bool on_diagonal = sub < heads_here && n0 / dh == sub;
    const __nv_bfloat16 *W = (g ? Wx : Wa) + ((size_t)h * k + sub) * dh * dh + (size_t)(o0 - sub * dh) * dh + (n0 - sub * dh);
    __half *W16m = W16 + ((size_t)g * H + h) * DH * DH;
#pragma unroll
    for (int r = threadIdx.y; r < 32; r += 8) {
        const float v = on_diagonal ? __bfloat162float(W[(size_t)r * dh + threadIdx.x]) : 0.0f;
        const __half hv = __float2half_rn(fminf(fmaxf(v, -65504.0f), 65504.0f));
        W16m[(size_t)(o0 + r) * DH + n0 + threadIdx.x] = hv;
        tile[r][threadIdx.x] = hv;
    }
    __syncthreads();
#pragma unroll
    for (int r = threadIdx.y; r < 32; r += 8)
        WT[((size_t)h * DH + n0 + r) * (2 * DH) + g * DH + o0 + threadIdx.x] = tile[threadIdx.x][r];
}

// Fixed-order sum over the token splits of the diagonal blocks of the groups' 256 x 256 weight gradients: one thread per
// element of dW_a / dW_x [H_layer][dh][dh].  part: [S][2 gates][G groups][256][256]
__global__ void reduce_dw_blocks_kernel(const float *part, int S, int G, int dh, int Hl, float *dWa, float *dWx) {
    const size_t per_gate = (size_t)Hl * dh * dh;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 2 * per_gate) return;
    const int gate = (int)(i / per_gate);
    size_t r = i % per_gate;
    const int n = (int)(r % dh); r /= dh;
    const int o = (int)(r % dh); r /= dh;
    const int head = (int)r, group = head / (DH / dh), sub = head % (DH / dh);
    const size_t src = (((size_t)gate * G + group) * DH + sub * dh + o) * DH + sub * dh + n;
    const size_t stride = (size_t)2 * G * DH * DH;
    float acc = 0.0f;
    for (int s = 0; s < S; ++s) acc += part[(size_t)s * stride + src];
    (gate ? dWx : dWa)[i % per_gate] = acc;
}

__device__ __forceinline__ __half to_half_sat(float v) { return __float2half_rn(fminf(fmaxf(v, -65504.0f), 65504.0f)); }

// u_t = b_c + sum_j w[j] x_{t-j}: one thread per (sequence, chunk, channel), forward in time.  grid (D/256, nchunk, B)
__global__ void __launch_bounds__(256) conv_forward_kernel(EwArgs a) {
    const int d = blockIdx.x * 256 + threadIdx.x, c = blockIdx.y, b = blockIdx.z;
    const int T = a.T, D = a.D;
    if (d >= D) return;
    const int t0 = c * CHUNK, t1 = min(T, t0 + CHUNK);
    float w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = bf2f(a.conv_w[(size_t)j * D + d]);
    const float cb = a.conv_b ? a.conv_b[d] : 0.0f;
    auto xat = [&](int t) -> float {
        if (t >= 0) return bf2f(a.x[((size_t)b * T + t) * D + d]);
        return a.cs_in ? bf2f(a.cs_in[((size_t)b * 3 + (3 + t)) * D + d]) : 0.0f;
    };
    float x3 = xat(t0 - 3), x2 = xat(t0 - 2), x1 = xat(t0 - 1);
    // eight tokens at a time, all loads first: u token-major (coalesced across the block)
    const uint32_t sD = (uint32_t)D;   // token stride; sixteen tokens' worth fits 32 bits
    auto batch8 = [&](__half *pu, const float (&xs)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float uv = fmaf(w[3], x3, fmaf(w[2], x2, fmaf(w[1], x1, fmaf(w[0], xs[k], cb))));
            pu[k * sD] = to_half_sat(uv);
            x3 = x2; x2 = x1; x1 = xs[k];
        }
    };
    int t = t0;
    for (; t + 16 <= t1; t += 16) {
        float xa[8], xb[8];
        const __nv_bfloat16 *px = a.x + ((size_t)b * T + t) * D + d;
        __half *pu = a.u + ((size_t)b * T + t) * D + d;
#pragma unroll
        for (int k = 0; k < 8; ++k) { xa[k] = bf2f(px[k * sD]); xb[k] = bf2f(px[(8 + k) * sD]); }
        batch8(pu, xa);
        batch8(pu + 8 * (size_t)sD, xb);
    }
    if (t < t1) {
        float xa[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) xa[k] = bf2f(a.x[((size_t)b * T + t + k) * D + d]);
        batch8(a.u + ((size_t)b * T + t) * D + d, xa);
    }
}

// Reverse scan, pass 1: per chunk the product of a_t and the carry a_first g_first it hands to earlier tokens when
// nothing comes in from later ones.  grid (D/256, nchunk, B)
__global__ void __launch_bounds__(256) scan_fold_kernel(EwArgs a) {
    const int d = blockIdx.x * 256 + threadIdx.x, c = blockIdx.y, b = blockIdx.z;
    if (d >= a.D) return;
    const int T = a.T, D = a.D, h = d / a.hstride, n = d % a.hstride;   // group of heads and channel slot within it
    const int t0 = c * CHUNK, t1 = min(T, t0 + CHUNK);
    const float s = decay_rate(a.lambda[d], a.c), ba = a.b_a[d];
    float carry = 0.0f, Q = 1.0f;
    const size_t tokb = (size_t)b * T + (t1 - 8);
    const uint32_t sD = (uint32_t)D, sZ = (uint32_t)a.H * 2 * DH;
    const __nv_bfloat16 *p_dy = a.dy + tokb * (size_t)sD + d;
    const __half *p_z = a.z + tokb * sZ + (size_t)h * 2 * DH + n;
    int tb = t1 - 8;
    // the kernel waits on memory: 16-token rounds keep 32 loads per thread in flight at 60 registers (32-token rounds
    // need 128 and measured the same); the pointers sit 8 tokens below the top of the round
    for (; tb - 8 >= t0; tb -= 16) {
        float dyv[16], zav[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) { dyv[k] = bf2f(p_dy[(k - 8) * (int)sD]); zav[k] = __half2float(p_z[(k - 8) * (int)sZ]); }
#pragma unroll
        for (int k = 15; k >= 0; --k) {
            const float at = __expf(-s * sigmoid_fast(zav[k] + ba));
            const float g = dyv[k] + carry;
            carry = at * g;
            Q *= at;
        }
        p_dy -= 16 * (size_t)sD; p_z -= 16 * (size_t)sZ;
    }
    for (; tb >= t0; tb -= 8) {
        float dyv[8], zav[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { dyv[k] = bf2f(p_dy[k * sD]); zav[k] = __half2float(p_z[k * sZ]); }
#pragma unroll
        for (int k = 7; k >= 0; --k) {
            const float at = __expf(-s * sigmoid_fast(zav[k] + ba));
            const float g = dyv[k] + carry;
            carry = at * g;
            Q *= at;
        }
        p_dy -= 8 * (size_t)sD; p_z -= 8 * (size_t)sZ;
    }
    a.fold[((size_t)b * a.nchunk + c) * D + d] = make_float2(Q, carry);
}

// pass 2: carries across chunks, last chunk first.  grid (D/256, B)
__global__ void __launch_bounds__(256) scan_carry_kernel(EwArgs a) {
    const int d = blockIdx.x * 256 + threadIdx.x, b = blockIdx.y;
    if (d >= a.D) return;
    // what later tokens hand to the last chunk: the gradient arriving on h_T (h_T = h_{T-1}, factor 1), else nothing
    float X = a.dh_T ? a.dh_T[(size_t)b * a.D + d] : 0.0f;
    // sixteen folds are requested at once (loads interleaved with the stores below would go out one at a time)
    for (int c1 = a.nchunk; c1 > 0; c1 -= 16) {
        float2 f[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int c = c1 - 1 - j;
            f[j] = c >= 0 ? a.fold[((size_t)b * a.nchunk + c) * a.D + d] : make_float2(1.0f, 0.0f);
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int c = c1 - 1 - j;
            if (c >= 0) {
                a.xin[((size_t)b * a.nchunk + c) * a.D + d] = X;
                X = fmaf(f[j].x, X, f[j].y);
            }
        }
    }
    if (a.dh0) a.dh0[(size_t)b * a.D + d] = X;   // what the first chunk hands on is a_0 g_0, the gradient of h0
}

// pass 3: the scan with its carry and every element-wise adjoint (derived from Eq. 1-4):
//   g_t = dy_t + a_{t+1} g_{t+1};  dL = g a (h_{t-1} - a v / m);  dv = g m;  di = dv u;  du = dv i;
//   dr = -s dL;  dz_a = dr r (1-r);  dz_x = di i (1-i);  dLambda += dL c r sigmoid(-Lambda).   grid (D/256, nchunk, B)
__global__ void __launch_bounds__(256, 3) scan_apply_kernel(EwArgs a) {
    const int d = blockIdx.x * 256 + threadIdx.x, c = blockIdx.y, b = blockIdx.z;
    if (d >= a.D) return;
    const int T = a.T, D = a.D, h = d / a.hstride, n = d % a.hstride;   // group of heads and channel slot within it
    const int t0 = c * CHUNK, t1 = min(T, t0 + CHUNK);
    const float lam = a.lambda[d];
    const float s = decay_rate(lam, a.c), ba = a.b_a[d], bx = a.b_x[d];
    const float dsdlam_neg = a.c * sigmoid_acc(-lam);
    float carry = a.xin[((size_t)b * a.nchunk + c) * D + d];
    float s_lam = 0.0f, s_ba = 0.0f, s_bx = 0.0f;
    // running pointers at token t1 - 8 (the loop walks backwards in steps of eight tokens)
    const size_t tokb = (size_t)b * T + (t1 - 8);
    const uint32_t sD = (uint32_t)D, sZ = (uint32_t)a.H * 2 * DH;      // token strides of [tok][D] and [tok][H][2][256] arrays; eight tokens' worth fits 32 bits
    const __nv_bfloat16 *p_dy = a.dy + tokb * (size_t)sD + d, *p_y = a.y + (tokb - 1) * (size_t)sD + d;
    const __half *p_z = a.z + tokb * (size_t)sZ + (size_t)h * 2 * DH + n, *p_u = a.u + tokb * (size_t)sD + d;
    __half *p_dz = a.dz + tokb * (size_t)sZ + (size_t)h * 2 * DH + n;
    __half *p_du = a.du + tokb * (size_t)sD + d;
    const float h0v = a.h0 ? a.h0[(size_t)b * D + d] : 0.0f;
    // eight tokens at the running pointers, newest first
    auto batch8 = [&](int tb) {
        float dza_hi = 0.0f, dzx_hi = 0.0f;
        float dyv[8], hpv[8], zav[8], zxv[8], uv[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            dyv[k] = bf2f(p_dy[k * sD]);
            hpv[k] = (tb + k) > 0 ? bf2f(p_y[k * sD]) : h0v;
            zav[k] = __half2float(p_z[k * sZ]);
            zxv[k] = __half2float(p_z[k * sZ + DH]);
            uv[k] = __half2float(p_u[k * sD]);
        }
#pragma unroll
        for (int k = 7; k >= 0; --k) {
            const float r = sigmoid_fast(zav[k] + ba), gi = sigmoid_fast(zxv[k] + bx);
            const float L = -s * r, at = __expf(L), m2 = one_minus_exp(2.0f * L);
            const float rm = m2 > 0.0f ? rsqrt_fast(m2) : 0.0f, mt = m2 * rm;   // 1/sqrt(1 - a^2) and sqrt(1 - a^2) from one MUFU
            const float g = dyv[k] + carry;
            carry = at * g;
            const float v = gi * uv[k];
            const float dL = g * (at * hpv[k] - at * at * v * rm);
            const float dv = g * mt;
            const float dza = -s * dL * r * (1.0f - r), dzx = dv * uv[k] * gi * (1.0f - gi);
            s_lam = fmaf(dL * r, dsdlam_neg, s_lam);
            s_ba += dza; s_bx += dzx;
            p_du[k * sD] = to_half_sat(dv * gi);
            // tokens k (odd) and k - 1 share one packed conversion
            if (k & 1) { dza_hi = dza; dzx_hi = dzx; }
            else {
                const uint32_t wa = pack_f16_sat(dza, dza_hi), wx = pack_f16_sat(dzx, dzx_hi);
                p_dz[k * sZ] = __ushort_as_half((unsigned short)(wa & 0xFFFFu));
                p_dz[(k + 1) * sZ] = __ushort_as_half((unsigned short)(wa >> 16));
                p_dz[k * sZ + DH] = __ushort_as_half((unsigned short)(wx & 0xFFFFu));
                p_dz[(k + 1) * sZ + DH] = __ushort_as_half((unsigned short)(wx >> 16));
            }
        }
        p_dy -= 8 * (size_t)sD; p_y -= 8 * (size_t)sD; p_z -= 8 * (size_t)sZ; p_u -= 8 * (size_t)sD; p_dz -= 8 * (size_t)sZ; p_du -= 8 * (size_t)sD;
    };
    int tb = t1 - 8;
    // sixteen tokens per round: the loads of the second eight are requested while the first eight are worked on
    for (; tb - 8 >= t0; tb -= 16) {
        batch8(tb);
        batch8(tb - 8);
    }
    if (tb >= t0) batch8(tb);
    float *pv = a.part_vec + ((size_t)b * a.nchunk + c) * 3 * D + d;
    pv[0] = s_lam; pv[(size_t)D] = s_ba; pv[(size_t)2 * D] = s_bx;
}

// Conv1D adjoint: dx_t = sum_j w[j] du_{t+j} (t + j < T); per-chunk partial sums of dw[j] = sum_t du_t x_{t-j} and
// db_c = sum_t du_t.  One thread per (sequence, chunk, channel) walks forward with sliding windows, so that every du and
// every x is loaded once.  grid (D/256, nchunk, B)
struct ConvBwdArgs {
    int B, T, D, nchunk;
    const __nv_bfloat16 *x, *conv_w, *cs_in;
    const __half *du;
    __nv_bfloat16 *dx;
    float *part_conv;   // [B*nchunk][5][D]
};

__global__ void __launch_bounds__(256) conv_backward_kernel(ConvBwdArgs a) {
    const int d = blockIdx.x * 256 + threadIdx.x, c = blockIdx.y, b = blockIdx.z;
    const int T = a.T, D = a.D;
    if (d >= D) return;
    const int t0 = c * CHUNK, t1 = min(T, t0 + CHUNK);
    float w[4], sw[4] = {0.f, 0.f, 0.f, 0.f}, sb = 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = bf2f(a.conv_w[(size_t)j * D + d]);
    auto xat = [&](int t) -> float {
        if (t >= 0) return bf2f(a.x[((size_t)b * T + t) * D + d]);
        return a.cs_in ? bf2f(a.cs_in[((size_t)b * 3 + (3 + t)) * D + d]) : 0.0f;
    };
    auto duat = [&](int t) -> float { return t < T ? __half2float(a.du[((size_t)b * T + t) * D + d]) : 0.0f; };
    float x1 = xat(t0 - 1), x2 = xat(t0 - 2), x3 = xat(t0 - 3);     // x_{t-1}, x_{t-2}, x_{t-3}
    float g0 = duat(t0), g1 = duat(t0 + 1), g2 = duat(t0 + 2);     // du_t, du_{t+1}, du_{t+2}
    const uint32_t sD = (uint32_t)D;   // token stride; eleven tokens' worth fits 32 bits
    for (int tb = t0; tb < t1; tb += 8) {
        float xs[8], gs[8];
        const size_t row = ((size_t)b * T + tb) * D + d;
        const __nv_bfloat16 *px = a.x + row;
        const __half *pg = a.du + row;
        __nv_bfloat16 *pdx = a.dx + row;
        if (tb + 11 <= T) {
#pragma unroll
            for (int k = 0; k < 8; ++k) { xs[k] = bf2f(px[k * sD]); gs[k] = __half2float(pg[(k + 3) * sD]); }
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) { xs[k] = bf2f(px[k * sD]); gs[k] = duat(tb + k + 3); }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float g3 = gs[k], x0 = xs[k];
            pdx[k * sD] = __float2bfloat16_rn(fmaf(w[3], g3, fmaf(w[2], g2, fmaf(w[1], g1, w[0] * g0))));
            sw[0] = fmaf(g0, x0, sw[0]); sw[1] = fmaf(g0, x1, sw[1]); sw[2] = fmaf(g0, x2, sw[2]); sw[3] = fmaf(g0, x3, sw[3]);
            sb += g0;
            g0 = g1; g1 = g2; g2 = g3;
            x3 = x2; x2 = x1; x1 = x0;
        }
    }
    float *pc = a.part_conv + ((size_t)(b * a.nchunk + c) * 5) * D + d;
#pragma unroll
    for (int j = 0; j < 4; ++j) pc[(size_t)j * D] = sw[j];
    pc[(size_t)4 * D] = sb;
}

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

unsigned gemm_grid(const GemmArgs &g) {
    int dev = 0, nsm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || nsm <= 0) nsm = 148;
    const int ntiles = g.nx * g.ny * g.H;
    return (unsigned)(ntiles < nsm ? ntiles : nsm);
}

// 256-slot groups of k = 256 / width (rounded down) consecutive heads: the unit of the GEMMs
inline int groups_of_heads(int D, int H) { const int k = DH / (D / H); return (H + k - 1) / k; }

struct BwdLayout {
    size_t BT, BTp, off_u, off_z, off_dz, off_du, off_y, off_hT, off_cs, off_fold, off_xin, off_pvec, off_pconv, off_pdw,
        off_wt, off_w16, off_fws, total;
    int nchunk, nchunk_conv, S, kb_per_split;
};

BwdLayout bwd_layout(int B, int T, int D, int Hl) {
    BwdLayout L{};
    const int H = groups_of_heads(D, Hl);   // the GEMMs work on 256-slot groups of heads
    const size_t Dg = (size_t)H * DH;         // channel slots of all groups (>= D)
    L.BT = (size_t)B * T;
    L.BTp = (L.BT + 63) & ~(size_t)63;
    L.nchunk = (T + CHUNK - 1) / CHUNK;
    L.nchunk_conv = (T + GENERIC_BWD_CHUNK - 1) / GENERIC_BWD_CHUNK;
    const int kblocks = (int)(L.BTp / 64);
    L.S = kblocks < 8 ? kblocks : 8;
    L.kb_per_split = (kblocks + L.S - 1) / L.S;
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t at = o; o += up256(bytes); return at; };
    L.off_u = take(L.BT * D * 2);
    L.off_z = take(L.BT * Dg * 2 * 2);
    L.off_dz = take(L.BT * Dg * 2 * 2);
    L.off_du = take(L.BT * D * 2);
    L.off_y = take(L.BT * D * 2);
    L.off_hT = take((size_t)B * D * 4);
    L.off_cs = take((size_t)B * 3 * D * 2);
    L.off_fold = take((size_t)B * L.nchunk * D * 8);
    L.off_xin = take((size_t)B * L.nchunk * D * 4);
    L.off_pvec = take((size_t)B * L.nchunk * 3 * D * 4);
    L.off_pconv = take((size_t)B * L.nchunk * 5 * D * 4);
    L.off_pdw = take((size_t)L.S * 2 * H * DH * DH * 4);
    L.off_wt = take((size_t)H * DH * 2 * DH * 2);
    L.off_w16 = take((size_t)H * DH * 2 * DH * 2);
    L.off_fws = take(WS_HEADER_BYTES + sm100_prefill_workspace_bytes(B, T, D, Hl));
    L.total = o;
    return L;
}

}  // namespace

// Head width: any multiple of 32 up to 256.  k = 256 / width (rounded down) consecutive heads form a group of 256 channel slots
// whose weight matrix is block-diagonal; it is multiplied as a dense 256 x 256 matrix (convert_w_kernel writes the zeros),
// and only the diagonal blocks of its gradient are kept (reduce_dw_blocks_kernel).  Slots beyond k width do not exist: they
// read neighbouring channels against zero weights and nothing of them is written to du.
bool sm100_backward_supported(int B, int T, int D, int H, int io) {
    if (io != RGLRU_BF16 || B <= 0 || T <= 0 || H <= 0 || D % H != 0 || T % 8 != 0) return false;
    const int dh = D / H;
    return dh <= DH && dh % 32 == 0;
}

size_t sm100_backward_workspace_bytes(int B, int T, int D, int H) { return bwd_layout(B, T, D, H).total; }

cudaError_t sm100_backward(const FwdArgs &fwd, BwdArgs &q, const void *y_saved, void *ws_body, size_t ws_body_bytes, uint32_t *status,
                           cudaStream_t st) {
    const int B = q.B, T = q.T, D = q.D, dh = q.D / q.H;
    const int H = groups_of_heads(D, q.H);   // 256-slot groups of heads: the unit of the GEMMs and of the z / dz arrays
    const int hstride = (DH / dh) * dh;      // channels from one group to the next
    const BwdLayout L = bwd_layout(B, T, D, q.H);
    if (ws_body_bytes < L.total) return cudaErrorInvalidValue;
    static PerDeviceOptIn opt_in;
    cudaError_t e = opt_in.ensure(tc_gemm_kernel, (int)GEMM_SMEM_ALLOC);
    if (e != cudaSuccess) return e;
    char *ws = (char *)ws_body;
    __half *u = (__half *)(ws + L.off_u), *z = (__half *)(ws + L.off_z);
    __half *dz = (__half *)(ws + L.off_dz), *WT = (__half *)(ws + L.off_wt), *W16 = (__half *)(ws + L.off_w16);
    __half *du = (__half *)(ws + L.off_du);

    // 0. h_{t-1} comes from the forward output; run the forward when the caller kept none
    const void *y = y_saved;
    if (y == nullptr) {
        FwdArgs f = fwd;
        f.y = ws + L.off_y; f.h_T = (float *)(ws + L.off_hT); f.cs_out = ws + L.off_cs;
        f.status = status;
        char *fws = ws + L.off_fws;
        e = sm100_prefill(f, fws + WS_HEADER_BYTES, sm100_prefill_workspace_bytes(B, T, D, q.H), st);
        if (e != cudaSuccess) return e;
        y = f.y;
    }

    if ((size_t)H * DH != (size_t)D) {
        // Some channel slots of the groups do not exist.  Nothing writes their dz, and although their weights are zero a NaN
        // bit pattern left in the workspace would still poison du = dz W: clear dz once.
        if ((e = cudaMemsetAsync(dz, 0, L.BT * (size_t)H * DH * 2 * 2, st)) != cudaSuccess) return e;
    }

    EwArgs a{};
    a.B = B; a.T = T; a.D = D; a.H = H; a.nchunk = L.nchunk; a.c = q.c; a.hstride = hstride;
    a.x = (const __nv_bfloat16 *)q.x; a.conv_w = (const __nv_bfloat16 *)q.conv_w; a.cs_in = (const __nv_bfloat16 *)q.cs_in;
    a.dy = (const __nv_bfloat16 *)q.dy; a.y = (const __nv_bfloat16 *)y;
    a.conv_b = fwd.conv_b; a.b_a = fwd.b_a; a.b_x = fwd.b_x; a.lambda = q.lambda; a.h0 = fwd.h0;
    a.u = u; a.dz = dz; a.z = z; a.du = du;
    a.fold = (float2 *)(ws + L.off_fold); a.xin = (float *)(ws + L.off_xin); a.part_vec = (float *)(ws + L.off_pvec);
    a.dh_T = q.dh_T; a.dh0 = q.dh0;

    // 1. W^T for the du contraction, conv output
    convert_w_kernel<<<dim3(DH / 32, DH / 32, 2 * H), dim3(32, 8), 0, st>>>((const __nv_bfloat16 *)q.W_a, (const __nv_bfloat16 *)q.W_x, W16, WT, H, dh, q.H);
    const dim3 grid_ew((D + 255) / 256, L.nchunk, B);
    conv_forward_kernel<<<grid_ew, 256, 0, st>>>(a);

    GemmArgs g{};
    g.H = H; g.D = D; g.hstride = hstride; g.cvalid = hstride; g.status = status; g.spin_ns = g_spin_limit_ns;
    const unsigned mtiles = (unsigned)((L.BT + 127) / 128);
    const uint64_t BT = L.BT;
    // 2. z = u W^T per head and gate
    {
        const uint64_t da[3] = {(uint64_t)D, BT, 1}, sa[2] = {(uint64_t)D * 2, (uint64_t)D * BT * 2};   // u [tok][D]
        const uint32_t ba[3] = {64, 128, 1};
        const uint64_t db[3] = {DH, DH, (uint64_t)H}, sb[2] = {DH * 2, (uint64_t)DH * DH * 2};
        const uint32_t bb[3] = {64, 256, 1};
        if (!encode_map16_3d(&g.tm_a, u, da, sa, ba, true) || !encode_map16_3d(&g.tm_b0, W16, db, sb, bb, true) ||
            !encode_map16_3d(&g.tm_b1, W16 + (size_t)H * DH * DH, db, sb, bb, true))
            return cudaErrorNotSupported;
        g.mode = MODE_Z; g.kblocks = DH / 64; g.rows_valid = (int)BT; g.out = z;
        g.nx = (int)mtiles; g.ny = 2;
        tc_gemm_kernel<<<gemm_grid(g), GEMM_THREADS, GEMM_SMEM_ALLOC, st>>>(g);
    }
    // 3. reverse scan and element-wise adjoints
    scan_fold_kernel<<<grid_ew, 256, 0, st>>>(a);
    scan_carry_kernel<<<dim3((D + 255) / 256, B), 256, 0, st>>>(a);
    scan_apply_kernel<<<grid_ew, 256, 0, st>>>(a);
    // 4. du += dz W
    {
        const uint64_t da[3] = {2 * DH, (uint64_t)H, BT}, sa[2] = {2 * DH * 2, (uint64_t)H * 2 * DH * 2};
        const uint32_t ba[3] = {64, 1, 128};
        const uint64_t db[3] = {2 * DH, DH, (uint64_t)H}, sb[2] = {2 * DH * 2, (uint64_t)DH * 2 * DH * 2};
        const uint32_t bb[3] = {64, 256, 1};
        if (!encode_map16_3d(&g.tm_a, dz, da, sa, ba, true) || !encode_map16_3d(&g.tm_b0, WT, db, sb, bb, true)) return cudaErrorNotSupported;
        g.tm_b1 = g.tm_b0;
        g.mode = MODE_DU; g.kblocks = 2 * DH / 64; g.rows_valid = (int)BT; g.out = du;
        g.nx = (int)mtiles; g.ny = 1;
        tc_gemm_kernel<<<gemm_grid(g), GEMM_THREADS, GEMM_SMEM_ALLOC, st>>>(g);
    }
    // 5. dW = dz^T u, split over the tokens, then a fixed-order sum of the splits
    {
        const uint64_t da[3] = {2 * DH, (uint64_t)H, BT}, sa[2] = {2 * DH * 2, (uint64_t)H * 2 * DH * 2};   // dz [tok][h][gate, channel]
        const uint32_t ba[3] = {64, 1, 64};
        const uint64_t db[3] = {(uint64_t)D, BT, 1}, sb[2] = {(uint64_t)D * 2, (uint64_t)D * BT * 2};         // u [tok][D]
        const uint32_t bb[3] = {64, 64, 1};
        if (!encode_map16_3d(&g.tm_a, dz, da, sa, ba, true) || !encode_map16_3d(&g.tm_b0, u, db, sb, bb, true)) return cudaErrorNotSupported;
        g.tm_b1 = g.tm_b0;
        float *part = (float *)(ws + L.off_pdw);
        g.mode = MODE_DW; g.kblocks = L.kb_per_split; g.rows_valid = 2 * DH; g.out = part;
        g.nx = 4; g.ny = L.S;
        tc_gemm_kernel<<<gemm_grid(g), GEMM_THREADS, GEMM_SMEM_ALLOC, st>>>(g);
        const size_t wsz = (size_t)H * DH * DH;
        if (dh == DH) {   // one head per group: the partial sums already have the layout of dW
            if ((e = reduce_partials3(part, L.S, 2 * wsz, q.dW_a, wsz, q.dW_x, wsz, nullptr, 0, st)) != cudaSuccess) return e;
        } else {
            const size_t nout = (size_t)2 * q.H * dh * dh;
            reduce_dw_blocks_kernel<<<(unsigned)((nout + 255) / 256), 256, 0, st>>>(part, L.S, H, dh, q.H, q.dW_a, q.dW_x);
        }
    }
    // 6. per-channel sums, Conv1D adjoint
    const int nparts = B * L.nchunk;
    if ((e = reduce_partials3(a.part_vec, nparts, (size_t)3 * D, q.dlambda, D, q.db_a, D, q.db_x, D, st)) != cudaSuccess) return e;
    ConvBwdArgs cb{};
    cb.B = B; cb.T = T; cb.D = D; cb.nchunk = L.nchunk;
    cb.x = a.x; cb.conv_w = a.conv_w; cb.cs_in = a.cs_in; cb.du = du; cb.dx = (__nv_bfloat16 *)q.dx;
    cb.part_conv = (float *)(ws + L.off_pconv);
    conv_backward_kernel<<<grid_ew, 256, 0, st>>>(cb);
    if ((e = state_conv_grads(q, RGLRU_BF16, du, true, st)) != cudaSuccess) return e;   // after dx: it rewrites the rows conv_state_out copies
    if ((e = reduce_partials3(cb.part_conv, nparts, (size_t)5 * D, q.dconv_w, (size_t)4 * D, q.dconv_b, D, nullptr, 0, st)) != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace rglru
