// Shape-generic CUDA-core kernels for the RG-LRU temporal core: any head width up to
// GENERIC_MAX_DH, fp32 or bf16 io, accurate libm-grade transcendental functions.
// They serve the fp32 configuration, head widths without a tensor-core kernel, and the
// backward.  One block walks one (sequence, head) pair through time; the gate products
// W_a u, W_x u (Eq. 1-2) run on FP32 FMAs with the weights staged through shared memory.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "rglru_internal.h"

namespace rglru {
namespace {

constexpr int NT = 256;  // threads per block
constexpr int GT = 16;   // tokens (or sequences, for decode) per tile
constexpr int NB = 16;   // input channels per staged weight slab

__device__ __forceinline__ float ldf(const float *p, size_t i) { return p[i]; }
__device__ __forceinline__ float ldf(const __nv_bfloat16 *p, size_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void stf(float *p, size_t i, float v) { p[i] = v; }
__device__ __forceinline__ void stf(__nv_bfloat16 *p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

__device__ __forceinline__ float sigmoid_acc(float z) { return 1.0f / (1.0f + expf(-z)); }
// GeLU(v) = v Phi(v), the non-linearity on the second branch of the recurrent block (Section 2.3)
__device__ __forceinline__ float gelu(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678f)); }

// s = c * softplus(-Lambda) = -c log sigmoid(Lambda)   (Appendix A, with a = sigmoid(Lambda))
__device__ __forceinline__ float decay_rate(float lambda, float c) {
    float z = -lambda;
    float sp = z > 0.0f ? z + log1pf(expf(-z)) : log1pf(expf(z));
    return c * sp;
}
// a_t = exp(-s r), m_t = sqrt(1 - a_t^2) = sqrt(-expm1(-2 s r))   (Eq. 3-4)
__device__ __forceinline__ void decay(float s, float r, float &a, float &m) {
    float L = -s * r;
    a = expf(L);
    m = sqrtf(fmaxf(0.0f, -expm1f(2.0f * L)));
}

// acc_a[tt] += sum_n W_a[o][n] u_s[tt][n] (same for W_x) for this thread's output channel o.
// Weight slabs of NB input channels are staged through shared memory, transposed so that
// threads read consecutive words.  Every thread of the block must call this.
template <typename IOT>
__device__ __forceinline__ void gate_accumulate(const IOT *__restrict__ Wa, const IOT *__restrict__ Wx, int Dh, int ob,
                                                const float *u_s, float *w_s, float (&acc_a)[GT], float (&acc_x)[GT]) {
    const int tid = threadIdx.x;
    const int o = ob * NT + tid;
    constexpr int WS_STRIDE = NT + 1;
#pragma unroll
    for (int tt = 0; tt < GT; ++tt) { acc_a[tt] = 0.0f; acc_x[tt] = 0.0f; }
    for (int n0 = 0; n0 < Dh; n0 += NB) {
        __syncthreads();
        // slab W[ob*NT .. +NT)[n0 .. n0+NB): consecutive lanes read consecutive n of one row
        for (int idx = tid; idx < NT * NB; idx += NT) {
            int oo = idx / NB, nn = idx % NB;
            int orow = ob * NT + oo, n = n0 + nn;
            float va = 0.0f, vx = 0.0f;
            if (orow < Dh && n < Dh) {
                va = ldf(Wa, (size_t)orow * Dh + n);
                vx = ldf(Wx, (size_t)orow * Dh + n);
            }
            w_s[nn * WS_STRIDE + oo] = va;
            w_s[(NB + nn) * WS_STRIDE + oo] = vx;
        }
        __syncthreads();
        if (o < Dh) {
            const int nmax = min(NB, Dh - n0);
            for (int nn = 0; nn < nmax; ++nn) {
                float wa = w_s[nn * WS_STRIDE + tid], wx = w_s[(NB + nn) * WS_STRIDE + tid];
#pragma unroll
                for (int tt = 0; tt < GT; ++tt) {
                    float uv = u_s[tt * Dh + n0 + nn];
                    acc_a[tt] = fmaf(wa, uv, acc_a[tt]);
                    acc_x[tt] = fmaf(wx, uv, acc_x[tt]);
                }
            }
        }
    }
}

// x_{tau} of sequence b for tau in [-3, T): history comes from conv_state_in (oldest first) or is zero
template <typename IOT>
__device__ __forceinline__ float x_at(const IOT *x, const IOT *cs_in, int T, int D, int b, int tau, int d) {
    if (tau >= 0) return ldf(x, ((size_t)b * T + tau) * D + d);
    if (cs_in == nullptr) return 0.0f;
    return ldf(cs_in, ((size_t)b * 3 + (3 + tau)) * D + d);
}
template <typename IOT>
__device__ __forceinline__ IOT x_raw_at(const IOT *x, const IOT *cs_in, int T, int D, int b, int tau, int d) {
    if (tau >= 0) return x[((size_t)b * T + tau) * D + d];
    if (cs_in == nullptr) return IOT(0.0f);
    return cs_in[((size_t)b * 3 + (3 + tau)) * D + d];
}

// Forward over T tokens for one (head, sequence) per block.  grid = (H, B).
// Dynamic shared memory: u_s[GT][Dh] | h_s[Dh] | w_s[2*NB][NT+1].
template <typename IOT, bool SAVE>
__global__ void __launch_bounds__(NT) generic_prefill_kernel(FwdArgs a) {
    extern __shared__ float smem[];
    const int Dh = a.D / a.H, D = a.D, T = a.T;
    const int k = blockIdx.x, b = blockIdx.y, d0 = k * Dh, tid = threadIdx.x;
    float *u_s = smem, *h_s = u_s + GT * Dh, *w_s = h_s + Dh;
    const IOT *x = (const IOT *)a.x, *cw = (const IOT *)a.conv_w, *cs_in = (const IOT *)a.cs_in;
    const IOT *Wa = (const IOT *)a.W_a + (size_t)k * Dh * Dh, *Wx = (const IOT *)a.W_x + (size_t)k * Dh * Dh;
    IOT *y = (IOT *)a.y;
    const IOT *gb = (const IOT *)a.gate_branch;
    const int nob = (Dh + NT - 1) / NT;

    for (int n = tid; n < Dh; n += NT) h_s[n] = a.h0 ? a.h0[(size_t)b * D + d0 + n] : 0.0f;

    for (int t0 = 0; t0 < T; t0 += GT) {
        const int len = min(GT, T - t0);
        __syncthreads();
        // Conv1D, width 4, causal: u_t = b_c + sum_j w[j] x_{t-j}
        for (int idx = tid; idx < GT * Dh; idx += NT) {
            int tt = idx / Dh, n = idx % Dh, d = d0 + n;
            float u = 0.0f;
            if (tt < len) {
                u = a.conv_b ? a.conv_b[d] : 0.0f;
#pragma unroll
                for (int j = 0; j < 4; ++j) u = fmaf(ldf(cw, (size_t)j * D + d), x_at(x, cs_in, T, D, b, t0 + tt - j, d), u);
                if (SAVE) a.save_u[((size_t)b * T + t0 + tt) * D + d] = u;
            }
            u_s[tt * Dh + n] = u;
        }
        __syncthreads();
        for (int ob = 0; ob < nob; ++ob) {
            float acc_a[GT], acc_x[GT];
            gate_accumulate<IOT>(Wa, Wx, Dh, ob, u_s, w_s, acc_a, acc_x);
            const int o = ob * NT + tid;
            if (o < Dh) {
                const int d = d0 + o;
                const float s = decay_rate(a.lambda[d], a.c), ba = a.b_a[d], bx = a.b_x[d];
                float h = h_s[o];
                // prod_t a_t of the call, carried from one time group to the next in the output itself (same thread each time)
                float ap = (a.a_prod && t0 > 0) ? a.a_prod[(size_t)b * D + d] : 1.0f;
#pragma unroll
                for (int tt = 0; tt < GT; ++tt) {
                    if (tt < len) {
                        float r = sigmoid_acc(acc_a[tt] + ba), g = sigmoid_acc(acc_x[tt] + bx), at, mt;
                        decay(s, r, at, mt);
                        size_t e = ((size_t)b * T + t0 + tt) * D + d;
                        if (SAVE) { a.save_r[e] = r; a.save_i[e] = g; a.save_hprev[e] = h; }
                        h = fmaf(at, h, mt * (g * u_s[tt * Dh + o]));
                        ap *= at;
                        // merged output of the recurrent block (Section 2.3): GeLU on the second branch, then the product
                        if (!SAVE) stf(y, e, gb ? h * gelu(ldf(gb, e)) : h);
                    }
                }
                h_s[o] = h;
                if (!SAVE && a.a_prod) a.a_prod[(size_t)b * D + d] = ap;
            }
        }
    }
    __syncthreads();
    if (!SAVE) {
        for (int n = tid; n < Dh; n += NT) a.h_T[(size_t)b * D + d0 + n] = h_s[n];
        // conv_state_out = last three raw inputs of concat(conv_state_in, x); staged so that it may alias conv_state_in
        IOT *stage = (IOT *)u_s;
        for (int idx = tid; idx < 3 * Dh; idx += NT) {
            int kk = idx / Dh, n = idx % Dh;
            stage[idx] = x_raw_at(x, cs_in, T, D, b, T - 3 + kk, d0 + n);
        }
        __syncthreads();
        IOT *cs_out = (IOT *)a.cs_out;
        for (int idx = tid; idx < 3 * Dh; idx += NT) {
            int kk = idx / Dh, n = idx % Dh;
            cs_out[((size_t)b * 3 + kk) * D + d0 + n] = stage[idx];
        }
    }
}

// One decode step.  grid = (H, ceil(B / GT)); a block handles GT sequences of one head.
template <typename IOT>
__global__ void __launch_bounds__(NT) generic_decode_kernel(FwdArgs a) {
    extern __shared__ float smem[];
    const int Dh = a.D / a.H, D = a.D, B = a.B;
    const int k = blockIdx.x, b0 = blockIdx.y * GT, d0 = k * Dh, tid = threadIdx.x;
    const int len = min(GT, B - b0);
    float *u_s = smem, *w_s = u_s + GT * Dh + Dh;
    const IOT *x = (const IOT *)a.x, *cw = (const IOT *)a.conv_w;
    IOT *cs = (IOT *)a.cs_out;  // in/out
    const IOT *Wa = (const IOT *)a.W_a + (size_t)k * Dh * Dh, *Wx = (const IOT *)a.W_x + (size_t)k * Dh * Dh;
    IOT *y = (IOT *)a.y;
    float *h = a.h_T;  // in/out
    const int nob = (Dh + NT - 1) / NT;

    for (int idx = tid; idx < GT * Dh; idx += NT) {
        int tt = idx / Dh, n = idx % Dh, d = d0 + n;
        float u = 0.0f;
        if (tt < len) {
            const int b = b0 + tt;
            IOT *c0 = cs + ((size_t)b * 3 + 0) * D + d, *c1 = c0 + D, *c2 = c1 + D;
            IOT r0 = *c0, r1 = *c1, r2 = *c2, xn = x[(size_t)b * D + d];
            u = a.conv_b ? a.conv_b[d] : 0.0f;
            u = fmaf(ldf(cw, (size_t)0 * D + d), ldf(&xn, 0), u);
            u = fmaf(ldf(cw, (size_t)1 * D + d), ldf(&r2, 0), u);
            u = fmaf(ldf(cw, (size_t)2 * D + d), ldf(&r1, 0), u);
            u = fmaf(ldf(cw, (size_t)3 * D + d), ldf(&r0, 0), u);
            *c0 = r1; *c1 = r2; *c2 = xn;  // bit-exact shift
        }
        u_s[tt * Dh + n] = u;
    }
    __syncthreads();
    for (int ob = 0; ob < nob; ++ob) {
        float acc_a[GT], acc_x[GT];
        gate_accumulate<IOT>(Wa, Wx, Dh, ob, u_s, w_s, acc_a, acc_x);
        const int o = ob * NT + tid;
        if (o < Dh) {
            const int d = d0 + o;
            const float s = decay_rate(a.lambda[d], a.c), ba = a.b_a[d], bx = a.b_x[d];
#pragma unroll
            for (int tt = 0; tt < GT; ++tt) {
                if (tt < len) {
                    float r = sigmoid_acc(acc_a[tt] + ba), g = sigmoid_acc(acc_x[tt] + bx), at, mt;
                    decay(s, r, at, mt);
                    size_t e = (size_t)(b0 + tt) * D + d;
                    float hn = fmaf(at, h[e], mt * (g * u_s[tt * Dh + o]));
                    h[e] = hn;
                    stf(y, e, hn);
                }
            }
        }
    }
}

// ------------------------------------------------------------------ backward
// Reverse-time scan and element-wise adjoints.  One thread per (b, d); grid = (ceil(D/NT), B).
//   g_t = dy_t + a_{t+1} g_{t+1};  dL = g (a h_{t-1} - a^2 v / m);  dv = g m;  di = dv u;  du = dv i;
//   dr = -s dL;  dz_a = dr r (1-r);  dz_x = di i (1-i).
// In place: r -> dz_a, i -> dz_x, hprev -> du (direct part).
template <typename IOT>
__global__ void __launch_bounds__(NT) generic_bwd_scan_kernel(BwdArgs q) {
    const int d = blockIdx.x * NT + threadIdx.x, b = blockIdx.y;
    if (d >= q.D) return;
    const int T = q.T, D = q.D;
    const IOT *dy = (const IOT *)q.dy;
    const float lam = q.lambda[d];
    const float s = decay_rate(lam, q.c);
    const float dsdlam_neg = q.c * sigmoid_acc(-lam);  // dL/dLambda = c r sigmoid(-Lambda)
    // past the last token g holds the gradient arriving on h_T (h_T = h_{T-1}, so it is carried with factor 1)
    float g = q.dh_T ? q.dh_T[(size_t)b * D + d] : 0.0f, a_next = 1.0f, s_lam = 0.0f, s_ba = 0.0f, s_bx = 0.0f;
    for (int t = T - 1; t >= 0; --t) {
        size_t e = ((size_t)b * T + t) * D + d;
        float r = q.r[e], gi = q.gi[e], u = q.u[e], hp = q.hp[e], at, mt;
        decay(s, r, at, mt);
        g = fmaf(a_next, g, ldf(dy, e));
        float v = gi * u;
        float dm_term = mt > 0.0f ? at * at * v / mt : 0.0f;
        float dL = g * (at * hp - dm_term);
        float dv = g * mt;
        float di = dv * u;
        float dr = -s * dL;
        float dza = dr * r * (1.0f - r), dzx = di * gi * (1.0f - gi);
        s_lam = fmaf(dL * r, dsdlam_neg, s_lam);
        s_ba += dza;
        s_bx += dzx;
        q.r[e] = dza;
        q.gi[e] = dzx;
        q.hp[e] = dv * gi;
        a_next = at;
    }
    if (q.dh0) q.dh0[(size_t)b * D + d] = a_next * g;   // a_0 g_0: h0 enters Eq. 4 only at t = 0
    q.part_vec[((size_t)b * 3 + 0) * D + d] = s_lam;
    q.part_vec[((size_t)b * 3 + 1) * D + d] = s_ba;
    q.part_vec[((size_t)b * 3 + 2) * D + d] = s_bx;
}

// du[tok][n] += sum_o W_a[o][n] dz_a[tok][o] + W_x[o][n] dz_x[tok][o].  grid = (H, ceil(B*T/GT)).
// Dynamic shared memory: dz_s[2][GT][Dh].
template <typename IOT>
__global__ void __launch_bounds__(NT) generic_bwd_du_kernel(BwdArgs q) {
    extern __shared__ float smem[];
    const int Dh = q.D / q.H, D = q.D, k = blockIdx.x, d0 = k * Dh, tid = threadIdx.x;
    const size_t ntok = (size_t)q.B * q.T, tok0 = (size_t)blockIdx.y * GT;
    const int len = (int)min((size_t)GT, ntok - tok0);
    float *dza_s = smem, *dzx_s = smem + GT * Dh;
    const IOT *Wa = (const IOT *)q.W_a + (size_t)k * Dh * Dh, *Wx = (const IOT *)q.W_x + (size_t)k * Dh * Dh;
    for (int idx = tid; idx < GT * Dh; idx += NT) {
        int tt = idx / Dh, o = idx % Dh;
        float va = 0.0f, vx = 0.0f;
        if (tt < len) { va = q.r[(tok0 + tt) * D + d0 + o]; vx = q.gi[(tok0 + tt) * D + d0 + o]; }
        dza_s[idx] = va; dzx_s[idx] = vx;
    }
    __syncthreads();
    for (int n = tid; n < Dh; n += NT) {
        float acc[GT];
#pragma unroll
        for (int tt = 0; tt < GT; ++tt) acc[tt] = 0.0f;
        for (int o = 0; o < Dh; ++o) {
            float wa = ldf(Wa, (size_t)o * Dh + n), wx = ldf(Wx, (size_t)o * Dh + n);
#pragma unroll
            for (int tt = 0; tt < GT; ++tt) acc[tt] = fmaf(wa, dza_s[tt * Dh + o], fmaf(wx, dzx_s[tt * Dh + o], acc[tt]));
        }
#pragma unroll
        for (int tt = 0; tt < GT; ++tt)
            if (tt < len) q.hp[(tok0 + tt) * D + d0 + n] += acc[tt];
    }
}

// Partial dW_a, dW_x: part[s][g][k][o][n] = sum over the tokens of split s of dz_g[tok][o] u[tok][n].
// grid = (H * ceil(Dh/GT), ceil(Dh/NT), S): a block owns GT output rows and NT input columns.
__global__ void __launch_bounds__(NT) generic_bwd_dw_kernel(BwdArgs q) {
    __shared__ float dz_s[2][GT][GT];
    const int Dh = q.D / q.H, D = q.D, tid = threadIdx.x;
    const int nobk = (Dh + GT - 1) / GT;
    const int k = blockIdx.x / nobk, o0 = (blockIdx.x % nobk) * GT, n = blockIdx.y * NT + tid, s = blockIdx.z;
    const int d0 = k * Dh;
    const size_t ntok = (size_t)q.B * q.T;
    const size_t per = (ntok + q.S - 1) / q.S;
    const size_t lo = (size_t)s * per, hi = min(ntok, lo + per);
    float acc_a[GT], acc_x[GT];
#pragma unroll
    for (int oo = 0; oo < GT; ++oo) { acc_a[oo] = 0.0f; acc_x[oo] = 0.0f; }
    for (size_t tok0 = lo; tok0 < hi; tok0 += GT) {
        __syncthreads();
        for (int idx = tid; idx < 2 * GT * GT; idx += NT) {
            int g = idx / (GT * GT), tt = (idx / GT) % GT, oo = idx % GT;
            float v = 0.0f;
            if (tok0 + tt < hi && o0 + oo < Dh) v = (g ? q.gi : q.r)[(tok0 + tt) * D + d0 + o0 + oo];
            dz_s[g][tt][oo] = v;
        }
        __syncthreads();
        if (n < Dh) {
            const int len = (int)min((size_t)GT, hi - tok0);
            for (int tt = 0; tt < len; ++tt) {
                float uv = q.u[(tok0 + tt) * D + d0 + n];
#pragma unroll
                for (int oo = 0; oo < GT; ++oo) {
                    acc_a[oo] = fmaf(dz_s[0][tt][oo], uv, acc_a[oo]);
                    acc_x[oo] = fmaf(dz_s[1][tt][oo], uv, acc_x[oo]);
                }
            }
        }
    }
    if (n < Dh) {
        const size_t wsz = (size_t)q.H * Dh * Dh;
#pragma unroll
        for (int oo = 0; oo < GT; ++oo) {
            if (o0 + oo < Dh) {
                size_t w = ((size_t)k * Dh + o0 + oo) * Dh + n;
                q.part_dw[((size_t)s * 2 + 0) * wsz + w] = acc_a[oo];
                q.part_dw[((size_t)s * 2 + 1) * wsz + w] = acc_x[oo];
            }
        }
    }
}

// Conv1D adjoint: dx_t = sum_j w[j] du_{t+j} (t+j < T); partial dw[j] = sum_t du_t x_{t-j}; partial db_c = sum_t du_t.
// One thread per (b, chunk, d); grid = (ceil(D/NT), nchunk, B).
template <typename IOT>
__global__ void __launch_bounds__(NT) generic_bwd_conv_kernel(BwdArgs q) {
    const int d = blockIdx.x * NT + threadIdx.x, ch = blockIdx.y, b = blockIdx.z;
    if (d >= q.D) return;
    const int T = q.T, D = q.D;
    const IOT *x = (const IOT *)q.x, *cs_in = (const IOT *)q.cs_in, *cw = (const IOT *)q.conv_w;
    IOT *dx = (IOT *)q.dx;
    float w[4], sw[4] = {0.f, 0.f, 0.f, 0.f}, sb = 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = ldf(cw, (size_t)j * D + d);
    const int t_lo = ch * GENERIC_BWD_CHUNK, t_hi = min(T, t_lo + GENERIC_BWD_CHUNK);
    for (int t = t_lo; t < t_hi; ++t) {
        float acc = 0.0f;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (t + j < T) acc = fmaf(w[j], q.hp[((size_t)b * T + t + j) * D + d], acc);
        stf(dx, ((size_t)b * T + t) * D + d, acc);
        float dut = q.hp[((size_t)b * T + t) * D + d];
#pragma unroll
        for (int j = 0; j < 4; ++j) sw[j] = fmaf(dut, x_at(x, cs_in, T, D, b, t - j, d), sw[j]);
        sb += dut;
    }
    float *p = q.part_conv + ((size_t)(b * q.nchunk + ch) * 5) * D + d;
#pragma unroll
    for (int j = 0; j < 4; ++j) p[(size_t)j * D] = sw[j];
    p[(size_t)4 * D] = sb;
}

// Gradient through the carried conv inputs and through the copies in conv_state_out.  One thread per (b, d); grid (ceil(D/NT), B).
template <typename IOT, typename DUT>
__global__ void __launch_bounds__(NT) state_conv_grads_kernel(BwdArgs q, const DUT *du) {
    const int d = blockIdx.x * NT + threadIdx.x, b = blockIdx.y;
    if (d >= q.D) return;
    const int T = q.T, D = q.D;
    const IOT *cw = (const IOT *)q.conv_w, *dcs_out = (const IOT *)q.dcs_out;
    IOT *dx = (IOT *)q.dx, *dcs_in = (IOT *)q.dcs_in;
    float w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = ldf(cw, (size_t)j * D + d);
    auto du_at = [&](int t) -> float { return (t >= 0 && t < T) ? (float)du[((size_t)b * T + t) * D + d] : 0.0f; };
    auto dxin = [&](int t) -> float {   // gradient of the conv input at time t (t may be negative): sum_j w[j] du_{t+j}
        float acc = 0.0f;
#pragma unroll
        for (int j = 0; j < 4; ++j) acc = fmaf(w[j], du_at(t + j), acc);
        return acc;
    };
    float in_grad[3];
#pragma unroll
    for (int r = 0; r < 3; ++r) in_grad[r] = dxin(r - 3);
    if (dcs_out) {
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            const float gk = ldf(dcs_out, ((size_t)b * 3 + k) * D + d);
            const int row = T + k;   // row of concat(conv_state_in, x) that conv_state_out[k] copies
            if (row >= 3) stf(dx, ((size_t)b * T + (row - 3)) * D + d, dxin(row - 3) + gk);
            else in_grad[row] += gk;
        }
    }
    if (dcs_in) {
#pragma unroll
        for (int r = 0; r < 3; ++r) stf(dcs_in, ((size_t)b * 3 + r) * D + d, in_grad[r]);
    }
}

// out[i] = sum_p in[p * stride + i], p ascending (fixed order => run-to-run identical results)
__global__ void reduce_partials_kernel(const float *in, int nparts, size_t stride, float *out, size_t n) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n || out == nullptr) return;
    float acc = 0.0f;
    for (int p = 0; p < nparts; ++p) acc += in[(size_t)p * stride + i];
    out[i] = acc;
}

// out[i] = sum over p of in[p * stride + i] in a fixed order (four interleaved running sums, added at the end), the row being
// split over three output arrays
__global__ void reduce_partials3_kernel(const float *in, int nparts, size_t stride, float *out0, size_t n0, float *out1, size_t n1,
                                        float *out2, size_t n2) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n0 + n1 + n2) return;
    float *out = i < n0 ? (out0 ? out0 + i : nullptr) : i < n0 + n1 ? (out1 ? out1 + (i - n0) : nullptr) : (out2 ? out2 + (i - n0 - n1) : nullptr);
    if (out == nullptr) return;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int p = 0;
    for (; p + 16 <= nparts; p += 16) {   // sixteen loads in flight, still four running sums in a fixed order
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = in[(size_t)(p + j) * stride + i];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j & 3] += v[j];
    }
    for (; p + 4 <= nparts; p += 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j] += in[(size_t)(p + j) * stride + i];
    }
    for (; p < nparts; ++p) acc[0] += in[(size_t)p * stride + i];
    *out = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

size_t fwd_smem_bytes(int Dh) { return sizeof(float) * ((size_t)GT * Dh + Dh + 2 * NB * (NT + 1)); }

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
    if (bytes > 48 * 1024) return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    return cudaSuccess;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

int dw_splits(size_t ntok) {
    size_t s = (ntok + 1023) / 1024;
    return (int)(s < 1 ? 1 : (s > 32 ? 32 : s));
}

}  // namespace

cudaError_t generic_prefill(const FwdArgs &a, int io, cudaStream_t st) {
    const int Dh = a.D / a.H;
    const size_t smem = fwd_smem_bytes(Dh);
    dim3 grid(a.H, a.B);
    cudaError_t e;
    const bool save = a.save_u != nullptr;
#define LAUNCH_PREFILL(IOT, SAVE)                                                     \
    do {                                                                              \
        if ((e = set_smem(generic_prefill_kernel<IOT, SAVE>, smem)) != cudaSuccess) return e; \
        generic_prefill_kernel<IOT, SAVE><<<grid, NT, smem, st>>>(a);                 \
    } while (0)
    if (io == RGLRU_F32) { if (save) LAUNCH_PREFILL(float, true); else LAUNCH_PREFILL(float, false); }
    else { if (save) LAUNCH_PREFILL(__nv_bfloat16, true); else LAUNCH_PREFILL(__nv_bfloat16, false); }
#undef LAUNCH_PREFILL
    return cudaGetLastError();
}

cudaError_t generic_decode(const FwdArgs &a, int io, cudaStream_t st) {
    const int Dh = a.D / a.H;
    const size_t smem = fwd_smem_bytes(Dh);
    dim3 grid(a.H, (a.B + GT - 1) / GT);
    cudaError_t e;
    if (io == RGLRU_F32) {
        if ((e = set_smem(generic_decode_kernel<float>, smem)) != cudaSuccess) return e;
        generic_decode_kernel<float><<<grid, NT, smem, st>>>(a);
    } else {
        if ((e = set_smem(generic_decode_kernel<__nv_bfloat16>, smem)) != cudaSuccess) return e;
        generic_decode_kernel<__nv_bfloat16><<<grid, NT, smem, st>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t state_conv_grads(const BwdArgs &q, int io, const void *du, bool du_is_half, cudaStream_t st) {
    if (!q.dcs_in && !q.dcs_out) return cudaSuccess;
    dim3 grid((q.D + NT - 1) / NT, q.B);
    if (io == RGLRU_F32) state_conv_grads_kernel<float, float><<<grid, NT, 0, st>>>(q, (const float *)du);
    else if (du_is_half) state_conv_grads_kernel<__nv_bfloat16, __half><<<grid, NT, 0, st>>>(q, (const __half *)du);
    else state_conv_grads_kernel<__nv_bfloat16, float><<<grid, NT, 0, st>>>(q, (const float *)du);
    return cudaGetLastError();
}

cudaError_t reduce_partials(const float *in, int nparts, size_t stride, float *out, size_t n, cudaStream_t st) {
    if (out == nullptr || n == 0) return cudaSuccess;
    reduce_partials_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(in, nparts, stride, out, n);
    return cudaGetLastError();
}

cudaError_t reduce_partials3(const float *in, int nparts, size_t stride, float *out0, size_t n0, float *out1, size_t n1, float *out2,
                             size_t n2, cudaStream_t st) {
    const size_t n = n0 + n1 + n2;
    if (n == 0 || (out0 == nullptr && out1 == nullptr && out2 == nullptr)) return cudaSuccess;
    reduce_partials3_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(in, nparts, stride, out0, n0, out1, n1, out2, n2);
    return cudaGetLastError();
}

size_t generic_backward_workspace_bytes(int B, int T, int D, int H) {
    const size_t btd = (size_t)B * T * D, Dh = D / H;
    const int nchunk = (T + GENERIC_BWD_CHUNK - 1) / GENERIC_BWD_CHUNK;
    const int S = dw_splits((size_t)B * T);
    size_t bytes = 4 * align256(btd * sizeof(float));
    bytes += align256((size_t)B * 3 * D * sizeof(float));
    bytes += align256((size_t)B * nchunk * 5 * D * sizeof(float));
    bytes += align256((size_t)S * 2 * H * Dh * Dh * sizeof(float));
    return bytes;
}

cudaError_t generic_backward(const FwdArgs &fwd_in, BwdArgs &q, int io, void *ws_body, cudaStream_t st) {
    const int B = q.B, T = q.T, D = q.D, H = q.H, Dh = D / H;
    const size_t btd = (size_t)B * T * D;
    char *p = (char *)ws_body;
    q.u = (float *)p; p += align256(btd * sizeof(float));
    q.r = (float *)p; p += align256(btd * sizeof(float));
    q.gi = (float *)p; p += align256(btd * sizeof(float));
    q.hp = (float *)p; p += align256(btd * sizeof(float));
    q.nchunk = (T + GENERIC_BWD_CHUNK - 1) / GENERIC_BWD_CHUNK;
    q.S = dw_splits((size_t)B * T);
    q.part_vec = (float *)p; p += align256((size_t)B * 3 * D * sizeof(float));
    q.part_conv = (float *)p; p += align256((size_t)B * q.nchunk * 5 * D * sizeof(float));
    q.part_dw = (float *)p;

    // 1. forward sweep, keeping u, r, i and h_{t-1} in fp32
    FwdArgs f = fwd_in;
    f.save_u = q.u; f.save_r = q.r; f.save_i = q.gi; f.save_hprev = q.hp;
    cudaError_t e = generic_prefill(f, io, st);
    if (e != cudaSuccess) return e;
    // 2. reverse-time scan + element-wise adjoints
    dim3 g2((D + NT - 1) / NT, B);
    if (io == RGLRU_F32) generic_bwd_scan_kernel<float><<<g2, NT, 0, st>>>(q);
    else generic_bwd_scan_kernel<__nv_bfloat16><<<g2, NT, 0, st>>>(q);
    // 3. du += W^T dz
    const size_t smem3 = sizeof(float) * 2 * GT * Dh;
    dim3 g3(H, (unsigned)((btd / D + GT - 1) / GT));
    if (io == RGLRU_F32) {
        if ((e = set_smem(generic_bwd_du_kernel<float>, smem3)) != cudaSuccess) return e;
        generic_bwd_du_kernel<float><<<g3, NT, smem3, st>>>(q);
    } else {
        if ((e = set_smem(generic_bwd_du_kernel<__nv_bfloat16>, smem3)) != cudaSuccess) return e;
        generic_bwd_du_kernel<__nv_bfloat16><<<g3, NT, smem3, st>>>(q);
    }
    // 4. dW partials and their reduction
    dim3 g4(H * ((Dh + GT - 1) / GT), (Dh + NT - 1) / NT, q.S);
    generic_bwd_dw_kernel<<<g4, NT, 0, st>>>(q);
    const size_t wsz = (size_t)H * Dh * Dh;
    reduce_partials_kernel<<<(unsigned)((wsz + 255) / 256), 256, 0, st>>>(q.part_dw, q.S, 2 * wsz, q.dW_a, wsz);
    reduce_partials_kernel<<<(unsigned)((wsz + 255) / 256), 256, 0, st>>>(q.part_dw + wsz, q.S, 2 * wsz, q.dW_x, wsz);
    // 5. Conv1D adjoint
    dim3 g5((D + NT - 1) / NT, q.nchunk, B);
    if (io == RGLRU_F32) generic_bwd_conv_kernel<float><<<g5, NT, 0, st>>>(q);
    else generic_bwd_conv_kernel<__nv_bfloat16><<<g5, NT, 0, st>>>(q);
    if ((e = state_conv_grads(q, io, q.hp, false, st)) != cudaSuccess) return e;   // after dx: it rewrites the rows conv_state_out copies
    // 6. deterministic reductions of the per-channel partial sums
    const unsigned gd = (D + 255) / 256;
    reduce_partials_kernel<<<gd, 256, 0, st>>>(q.part_vec, B, (size_t)3 * D, q.dlambda, D);
    reduce_partials_kernel<<<gd, 256, 0, st>>>(q.part_vec + D, B, (size_t)3 * D, q.db_a, D);
    reduce_partials_kernel<<<gd, 256, 0, st>>>(q.part_vec + 2 * (size_t)D, B, (size_t)3 * D, q.db_x, D);
    reduce_partials_kernel<<<(4 * D + 255) / 256, 256, 0, st>>>(q.part_conv, B * q.nchunk, (size_t)5 * D, q.dconv_w, (size_t)4 * D);
    reduce_partials_kernel<<<gd, 256, 0, st>>>(q.part_conv + 4 * (size_t)D, B * q.nchunk, (size_t)5 * D, q.dconv_b, D);
    return cudaGetLastError();
}

}  // namespace rglru
