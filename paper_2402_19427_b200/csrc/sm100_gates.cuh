// Gate, decay and input-scale arithmetic of Eq. 1-4 shared by the sm_100a forward kernels (prefill and decode), on
// packed fp32x2 registers.  Device code only.
#pragma once

#include "sm100_ptx.cuh"

namespace rglru {

// Channels whose decay rate s = c*softplus(-Lambda) is at most S_POLY evaluate exp on the FMA pipe.
constexpr float S_POLY = 0.25f;

using namespace ptx;

// (z_a, z_x) of two tokens (or two sequences) of one channel, one per half of each register pair -> (a_t, v_t) of Eq. 3-4,
// in place, for W register pairs advanced in lock step (independent dependency chains side by side).
//   r = sigmoid(z_a + b_a) = 1/2 + 1/2 tanh((z_a + b_a)/2),  x = 2 s r,  f = 1 - a_t = -expm1(-x/2),
//   m/2 = sqrt(f (1/2 - f/4)) = sqrt(1 - a_t^2)/2,  v = (m/2 u)(1 + tanh((z_x + b_x)/2)) = m i u.
template <bool POLY, int W>
__device__ __forceinline__ void gate_group(f32x2 *za, f32x2 *zx, const float *u, f32x2 hba2, f32x2 hbx2, f32x2 s2) {
    const f32x2 HALF2 = pack2(0.5f, 0.5f), NEG1 = pack2(-1.0f, -1.0f), ONE2 = pack2(1.0f, 1.0f);
    f32x2 ta[W], tx[W], x[W], f[W], q[W];
#pragma unroll
    for (int i = 0; i < W; ++i) { ta[i] = fma2(za[i], HALF2, hba2); tx[i] = fma2(zx[i], HALF2, hbx2); }
#pragma unroll
    for (int i = 0; i < W; ++i) ta[i] = pack2(tanh_approx(lo2(ta[i])), tanh_approx(hi2(ta[i])));
#pragma unroll
    for (int i = 0; i < W; ++i) tx[i] = pack2(tanh_approx(lo2(tx[i])), tanh_approx(hi2(tx[i])));
#pragma unroll
    for (int i = 0; i < W; ++i) x[i] = fma2(ta[i], s2, s2);
    if (POLY) {
        // f = x/2 - x^2/8 + x^3/48 - x^4/384  (|x| <= 2 S_POLY: relative truncation error < 4e-5)
        f32x2 p[W];
#pragma unroll
        for (int i = 0; i < W; ++i) p[i] = fma2(x[i], pack2(-1.0f / 384.0f, -1.0f / 384.0f), pack2(1.0f / 48.0f, 1.0f / 48.0f));
#pragma unroll
        for (int i = 0; i < W; ++i) p[i] = fma2(p[i], x[i], pack2(-0.125f, -0.125f));
#pragma unroll
        for (int i = 0; i < W; ++i) p[i] = fma2(p[i], x[i], HALF2);
#pragma unroll
        for (int i = 0; i < W; ++i) { f[i] = mul2(p[i], x[i]); za[i] = fma2(f[i], NEG1, ONE2); }
    } else {
#pragma unroll
        for (int i = 0; i < W; ++i) {
            const f32x2 e = mul2(x[i], pack2(-0.72134752f, -0.72134752f));  // -x/2 * log2(e)
            za[i] = pack2(ex2_approx(lo2(e)), ex2_approx(hi2(e)));
            f[i] = fma2(za[i], NEG1, ONE2);
        }
    }
#pragma unroll
    for (int i = 0; i < W; ++i) q[i] = mul2(f[i], fma2(f[i], pack2(-0.25f, -0.25f), HALF2));  // (1 - a^2)/4 = f (2 - f)/4
    if (!POLY) {
#pragma unroll
        for (int i = 0; i < W; ++i) q[i] = pack2(fmaxf(lo2(q[i]), 0.0f), fmaxf(hi2(q[i]), 0.0f));  // a from ex2.approx may round above 1
    }
#pragma unroll
    for (int i = 0; i < W; ++i) q[i] = pack2(sqrt_approx(lo2(q[i])), sqrt_approx(hi2(q[i])));
#pragma unroll
    for (int i = 0; i < W; ++i) { const f32x2 g = mul2(q[i], pack2(u[2 * i], u[2 * i + 1])); zx[i] = fma2(g, tx[i], g); }
}


}  // namespace rglru
