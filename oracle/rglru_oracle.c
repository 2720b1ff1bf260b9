/*
 * rglru_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, sequential-in-time fp64 statement of the temporal core of the
 * Griffin/Hawk recurrent block: causal depthwise Conv1D of temporal width 4
 * (Section 2.3, "Recurrent block") followed by the RG-LRU layer (Section 2.4,
 * Eq. 1-4), with the decay evaluated in log space (Appendix A) and the gate
 * matrices block-diagonal per head (Section 4.1, paragraph "Recurrent Block").
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * load this file.  It shares no code, header, table or helper with the CUDA
 * library and is never reached from the product path.
 *
 * Every tensor is a dense row-major array of doubles; callers convert the
 * stored fp32/bf16 values exactly.  Notation follows the paper: x_t is the
 * layer input, u_t the Conv1D output (the "x_t" seen by Eq. 1-4), r_t and i_t
 * the recurrence and input gates, a_t the decay, h_t the state, y_t = h_t.
 *
 * Readings where the text is silent or at odds with itself:
 *  - a = sigmoid(Lambda) (Section 2.4), hence log a_t = -c*softplus(-Lambda)*r_t.
 *    Appendix A prints softplus(+Lambda); that is the same layer under
 *    Lambda -> -Lambda and contradicts "a = sigmoid(Lambda)".
 *  - the conv is causal, tap j multiplies x_{t-j}, history before t=0 comes
 *    from conv_state_in (oldest first), else zero.
 *  - W[k][o][n]: head k, output channel o, input channel n ("W x").
 *  - sqrt(1-a_t^2) is evaluated as sqrt(-expm1(2 log a_t)), clamped at 0.
 *
 * Parity pins (tests/test_oracle_pins.py): closed form for constant gates,
 * unit stationary variance, zero input, linearity in h0, prefill == chained
 * decode == split prefill, causality / head / batch independence, textbook
 * conv1d + matmul + monoid-fold reconstruction, gate curves, Lambda init
 * values, central finite differences for the backward.  No function here is
 * "parity unpinned".
 *
 * Threading: OpenMP over independent (batch, head) units only; the time loop
 * is sequential.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define CONV_WIDTH 4

static double logistic(double z) { return 1.0 / (1.0 + exp(-z)); }

/* log(1 + e^z) without overflow */
static double softplus(double z) { return z > 0.0 ? z + log1p(exp(-z)) : log1p(exp(z)); }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Eq. 3 in log space (Appendix A): a_t = sigmoid(Lambda)^(c r_t), and the input
 * scale sqrt(1 - a_t^2) of Eq. 4.  Also the alpha(r), beta(r) curves of the
 * "Gate behaviour" paragraph of Appendix A. */
void oracle_decay(double lambda, double r, double c, double *a_t, double *m_t) {
    double s = c * softplus(-lambda); /* = -c log sigmoid(Lambda) >= 0 */
    double L = -s * r;                /* log a_t */
    double q = -expm1(2.0 * L);       /* 1 - a_t^2 */
    *a_t = exp(L);
    *m_t = sqrt(q > 0.0 ? q : 0.0);
}

/* x_{tau} for tau in [-3, T): history before the segment comes from conv_state_in
 * ([B,3,D], oldest first: row 0 = x_{-3}), or is zero. */
static double x_at(const double *x, const double *cs_in, int T, int D, int b, int tau, int d) {
    if (tau >= 0) return x[((size_t)b * T + tau) * D + d];
    if (cs_in == NULL) return 0.0;
    return cs_in[((size_t)b * 3 + (3 + tau)) * D + d];
}

/* Conv1D output u_t for one (b, t) over the channels of one head. */
static void conv_row(const double *x, const double *cs_in, const double *conv_w, const double *conv_b,
                     int T, int D, int b, int t, int d0, int Dh, double *u) {
    for (int n = 0; n < Dh; ++n) {
        int d = d0 + n;
        double acc = conv_b ? conv_b[d] : 0.0;
        for (int j = 0; j < CONV_WIDTH; ++j) acc += conv_w[(size_t)j * D + d] * x_at(x, cs_in, T, D, b, t - j, d);
        u[n] = acc;
    }
}

/* z = W[k] u + bias for one head: W[k] is [Dh][Dh], row = output channel. */
static void gate_preact(const double *Wk, const double *bias, const double *u, int Dh, double *z) {
    for (int o = 0; o < Dh; ++o) {
        double acc = bias[o];
        const double *row = Wk + (size_t)o * Dh;
        for (int n = 0; n < Dh; ++n) acc += row[n] * u[n];
        z[o] = acc;
    }
}

/* Last three raw inputs of concat(conv_state_in, x), oldest first. */
static void write_conv_state(const double *x, const double *cs_in, int B, int T, int D, double *cs_out) {
    double *tmp = (double *)malloc((size_t)B * 3 * D * sizeof(double));
    for (int b = 0; b < B; ++b)
        for (int k = 0; k < 3; ++k)
            for (int d = 0; d < D; ++d) tmp[((size_t)b * 3 + k) * D + d] = x_at(x, cs_in, T, D, b, T - 3 + k, d);
    memcpy(cs_out, tmp, (size_t)B * 3 * D * sizeof(double));
    free(tmp);
}

/* GeLU(v) = v Phi(v) with Phi the standard normal distribution function: the definition of the non-linearity the
 * recurrent block applies to its second branch (Section 2.3). */
double oracle_gelu(double v) { return 0.5 * v * (1.0 + erf(v / sqrt(2.0))); }

/*
 * Prefill / forward over T tokens.  Returns 0, or -1 on a bad shape.
 *   x [B,T,D]; conv_w [4,D]; conv_b [D] or NULL; W_a, W_x [H,Dh,Dh]; b_a, b_x, lambda [D];
 *   h0 [B,D] or NULL (zero); conv_state_in [B,3,D] or NULL (zero);
 *   y [B,T,D]; h_T [B,D] (may alias h0); conv_state_out [B,3,D] (may alias conv_state_in);
 *   gate_branch [B,T,D] or NULL: the second branch of the recurrent block (Section 2.3: GeLU on that branch, then the
 *       two branches are merged by element-wise multiplication).  With it y_t = h_t * GeLU(gate_branch_t); the
 *       carried state h_T stays the raw h;
 *   a_prod [B,D] or NULL, out: prod_t a_t over the T tokens.  Eq. 4 is affine in the incoming state, so
 *       h_T = a_prod * h0 + (h_T from a zero state): (a_prod, h_T from zero) describes the whole call as one step.
 */
int oracle_prefill(int B, int T, int D, int H, double c, const double *x, const double *conv_w, const double *conv_b,
                   const double *W_a, const double *b_a, const double *W_x, const double *b_x, const double *lambda,
                   const double *h0, const double *conv_state_in, double *y, double *h_T, double *conv_state_out,
                   const double *gate_branch, double *a_prod) {
    if (B <= 0 || T <= 0 || D <= 0 || H <= 0 || D % H != 0) return -1;
    const int Dh = D / H;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int k = 0; k < H; ++k) {
            const int d0 = k * Dh;
            double *u = (double *)malloc(sizeof(double) * Dh * 5);
            double *za = u + Dh, *zx = u + 2 * Dh, *h = u + 3 * Dh, *ap = u + 4 * Dh;
            for (int n = 0; n < Dh; ++n) { h[n] = h0 ? h0[(size_t)b * D + d0 + n] : 0.0; ap[n] = 1.0; }
            for (int t = 0; t < T; ++t) {
                conv_row(x, conv_state_in, conv_w, conv_b, T, D, b, t, d0, Dh, u);
                gate_preact(W_a + (size_t)k * Dh * Dh, b_a + d0, u, Dh, za); /* Eq. 1 */
                gate_preact(W_x + (size_t)k * Dh * Dh, b_x + d0, u, Dh, zx); /* Eq. 2 */
                for (int n = 0; n < Dh; ++n) {
                    double r = logistic(za[n]), i = logistic(zx[n]), a, m;
                    const size_t at = ((size_t)b * T + t) * D + d0 + n;
                    oracle_decay(lambda[d0 + n], r, c, &a, &m);  /* Eq. 3 */
                    h[n] = a * h[n] + m * (i * u[n]);            /* Eq. 4 */
                    ap[n] *= a;
                    y[at] = gate_branch ? h[n] * oracle_gelu(gate_branch[at]) : h[n];  /* y_t = h_t [merged, Section 2.3] */
                }
            }
            /* h_T may alias h0: each (b, head) slice is read above before it is written here */
            for (int n = 0; n < Dh; ++n) h_T[(size_t)b * D + d0 + n] = h[n];
            if (a_prod)
                for (int n = 0; n < Dh; ++n) a_prod[(size_t)b * D + d0 + n] = ap[n];
            free(u);
        }
    }
    write_conv_state(x, conv_state_in, B, T, D, conv_state_out);
    return 0;
}

/*
 * One decode step for B sequences (Appendix F.4, "Cache sizes": the carried state is h, size D_RNN,
 * and the last 4-1 = 3 conv inputs).  Written from the state definition, not by calling
 * the prefill: h [B,D] and conv_state [B,3,D] are updated in place, y [B,D] is written.
 */
int oracle_decode_step(int B, int D, int H, double c, const double *x, const double *conv_w, const double *conv_b,
                       const double *W_a, const double *b_a, const double *W_x, const double *b_x,
                       const double *lambda, double *h, double *conv_state, double *y) {
    if (B <= 0 || D <= 0 || H <= 0 || D % H != 0) return -1;
    const int Dh = D / H;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int k = 0; k < H; ++k) {
            const int d0 = k * Dh;
            double *u = (double *)malloc(sizeof(double) * Dh * 3);
            double *za = u + Dh, *zx = u + 2 * Dh;
            double *cs = conv_state + (size_t)b * 3 * D;
            for (int n = 0; n < Dh; ++n) {
                int d = d0 + n;
                double xn = x[(size_t)b * D + d];
                /* window (x_{t-3}, x_{t-2}, x_{t-1}, x_t) = (cs[0], cs[1], cs[2], xn); tap j hits x_{t-j} */
                u[n] = (conv_b ? conv_b[d] : 0.0) + conv_w[0 * (size_t)D + d] * xn + conv_w[1 * (size_t)D + d] * cs[2 * (size_t)D + d] +
                       conv_w[2 * (size_t)D + d] * cs[1 * (size_t)D + d] + conv_w[3 * (size_t)D + d] * cs[0 * (size_t)D + d];
                /* shift the window: drop the oldest, append the new input */
                cs[0 * (size_t)D + d] = cs[1 * (size_t)D + d];
                cs[1 * (size_t)D + d] = cs[2 * (size_t)D + d];
                cs[2 * (size_t)D + d] = xn;
            }
            gate_preact(W_a + (size_t)k * Dh * Dh, b_a + d0, u, Dh, za);
            gate_preact(W_x + (size_t)k * Dh * Dh, b_x + d0, u, Dh, zx);
            for (int n = 0; n < Dh; ++n) {
                double r = logistic(za[n]), i = logistic(zx[n]), a, m;
                oracle_decay(lambda[d0 + n], r, c, &a, &m);
                double hn = a * h[(size_t)b * D + d0 + n] + m * (i * u[n]);
                h[(size_t)b * D + d0 + n] = hn;
                y[(size_t)b * D + d0 + n] = hn;
            }
            free(u);
        }
    }
    return 0;
}

/*
 * Backward of oracle_prefill for the scalar
 *     loss = sum(dy * y) + sum(dh_T * h_T) + sum(dconv_state_out * conv_state_out)
 * (the last two terms only when the pointers are given: they are what flows back from a later segment of the same sequence
 * through the state this segment handed on, so that a sequence can be differentiated segment by segment).  The paper gives
 * no backward; this is reverse-mode differentiation of Eq. 1-4 and of the Conv1D, written out:
 *
 *   g_t   = dy_t + a_{t+1} g_{t+1}                     (adjoint of h_t; beyond the last token g is dh_T, carried with factor 1
 *                                                       because h_T = h_{T-1}; 0 when dh_T is not given)
 *   dL_t  = g_t (a_t h_{t-1} - a_t^2 v_t / m_t)        (L_t = log a_t, v_t = i_t u_t, m_t = sqrt(1-a_t^2);
 *                                                       the second term is taken as 0 when m_t = 0)
 *   dv_t  = g_t m_t ;  di_t = dv_t u_t ;  du_t += dv_t i_t
 *   dr_t  = -s dL_t  with s = c softplus(-Lambda);  dLambda += dL_t c r_t sigmoid(-Lambda)
 *   dz_a  = dr r (1-r) ;  dz_x = di i (1-i) ;  db += dz ;  dW[k][o][n] += dz[o] u[n]
 *   du_t += W_a[k]^T dz_a + W_x[k]^T dz_x
 *   dx_t  = sum_j w[j] du_{t+j} (t+j < T) ;  dw[j] += du_t x_{t-j} ;  db_c += du_t
 *   dh0   = a_0 g_0                                    (h_{-1} = h0 enters Eq. 4 only at t = 0)
 *   dconv_state_in[r] = sum_j w[j] du_{r-3+j} (0 <= r-3+j < T)      (row r is x_{r-3}: the same formula as dx, at t < 0)
 *   conv_state_out is a copy of the last three rows of concat(conv_state_in, x): dconv_state_out[k] is added to the
 *   gradient of that row (dx_{T-3+k}, or dconv_state_in[T+k] when T+k < 3).
 *
 * All parameter gradients are overwritten (summed over batch and time).
 *   dx [B,T,D]; dconv_w [4,D]; dconv_b [D] (or NULL to skip); dW_a, dW_x [H,Dh,Dh]; db_a, db_x, dlambda [D].
 *   dh_T [B,D], dconv_state_out [B,3,D]: in, or NULL for zero.  dh0 [B,D], dconv_state_in [B,3,D]: out, or NULL to skip.
 */
int oracle_backward(int B, int T, int D, int H, double c, const double *x, const double *conv_w, const double *conv_b,
                    const double *W_a, const double *b_a, const double *W_x, const double *b_x, const double *lambda,
                    const double *h0, const double *conv_state_in, const double *dy, double *dx, double *dconv_w,
                    double *dconv_b, double *dW_a, double *db_a, double *dW_x, double *db_x, double *dlambda,
                    const double *dh_T, const double *dconv_state_out, double *dh0, double *dconv_state_in) {
    if (B <= 0 || T <= 0 || D <= 0 || H <= 0 || D % H != 0) return -1;
    const int Dh = D / H;
    memset(dconv_w, 0, sizeof(double) * 4 * D);
    if (dconv_b) memset(dconv_b, 0, sizeof(double) * D);
    memset(dW_a, 0, sizeof(double) * (size_t)H * Dh * Dh);
    memset(dW_x, 0, sizeof(double) * (size_t)H * Dh * Dh);
    memset(db_a, 0, sizeof(double) * D);
    memset(db_x, 0, sizeof(double) * D);
    memset(dlambda, 0, sizeof(double) * D);
    /* heads are independent; the batch loop is inside so that each thread owns its head's accumulators */
#pragma omp parallel for schedule(dynamic)
    for (int k = 0; k < H; ++k) {
        const int d0 = k * Dh;
        const size_t TD = (size_t)T * Dh;
        double *u = (double *)malloc(sizeof(double) * TD * 7);
        double *r = u + TD, *gi = u + 2 * TD, *a = u + 3 * TD, *m = u + 4 * TD, *hprev = u + 5 * TD, *du = u + 6 * TD;
        double *za = (double *)malloc(sizeof(double) * Dh * 5);
        double *zx = za + Dh, *h = za + 2 * Dh, *g = za + 3 * Dh, *dza = za + 4 * Dh;
        double *dzx = (double *)malloc(sizeof(double) * Dh);
        const double *Wak = W_a + (size_t)k * Dh * Dh, *Wxk = W_x + (size_t)k * Dh * Dh;
        for (int b = 0; b < B; ++b) {
            /* forward sweep, keeping what the reverse sweep needs */
            for (int n = 0; n < Dh; ++n) h[n] = h0 ? h0[(size_t)b * D + d0 + n] : 0.0;
            for (int t = 0; t < T; ++t) {
                double *ut = u + (size_t)t * Dh;
                conv_row(x, conv_state_in, conv_w, conv_b, T, D, b, t, d0, Dh, ut);
                gate_preact(Wak, b_a + d0, ut, Dh, za);
                gate_preact(Wxk, b_x + d0, ut, Dh, zx);
                for (int n = 0; n < Dh; ++n) {
                    size_t e = (size_t)t * Dh + n;
                    r[e] = logistic(za[n]);
                    gi[e] = logistic(zx[n]);
                    oracle_decay(lambda[d0 + n], r[e], c, &a[e], &m[e]);
                    hprev[e] = h[n];
                    h[n] = a[e] * h[n] + m[e] * (gi[e] * ut[n]);
                }
            }
            /* reverse sweep */
            for (int n = 0; n < Dh; ++n) g[n] = dh_T ? dh_T[(size_t)b * D + d0 + n] : 0.0;
            for (int t = T - 1; t >= 0; --t) {
                double *ut = u + (size_t)t * Dh, *dut = du + (size_t)t * Dh;
                for (int n = 0; n < Dh; ++n) {
                    size_t e = (size_t)t * Dh + n;
                    int d = d0 + n;
                    double a_next = (t + 1 < T) ? a[e + Dh] : 1.0;   /* past the end g holds dh_T (or 0) */
                    g[n] = dy[((size_t)b * T + t) * D + d] + a_next * g[n];
                    double v = gi[e] * ut[n];
                    double dm_term = (m[e] > 0.0) ? a[e] * a[e] * v / m[e] : 0.0;
                    double dL = g[n] * (a[e] * hprev[e] - dm_term);
                    double dv = g[n] * m[e];
                    double di = dv * ut[n];
                    dut[n] = dv * gi[e];
                    double s = c * softplus(-lambda[d]);
                    double dr = -s * dL;
                    dlambda[d] += dL * c * r[e] * logistic(-lambda[d]);
                    dza[n] = dr * r[e] * (1.0 - r[e]);
                    dzx[n] = di * gi[e] * (1.0 - gi[e]);
                    db_a[d] += dza[n];
                    db_x[d] += dzx[n];
                }
                for (int o = 0; o < Dh; ++o) {
                    double *dWa_row = dW_a + ((size_t)k * Dh + o) * Dh, *dWx_row = dW_x + ((size_t)k * Dh + o) * Dh;
                    const double *Wa_row = Wak + (size_t)o * Dh, *Wx_row = Wxk + (size_t)o * Dh;
                    for (int n = 0; n < Dh; ++n) {
                        dWa_row[n] += dza[o] * ut[n];
                        dWx_row[n] += dzx[o] * ut[n];
                        dut[n] += Wa_row[n] * dza[o] + Wx_row[n] * dzx[o];
                    }
                }
            }
            if (dh0)
                for (int n = 0; n < Dh; ++n) dh0[(size_t)b * D + d0 + n] = a[n] * g[n];   /* a_0 g_0 */
            /* Conv1D backward */
            for (int t = 0; t < T; ++t) {
                for (int n = 0; n < Dh; ++n) {
                    int d = d0 + n;
                    double acc = 0.0;
                    for (int j = 0; j < CONV_WIDTH && t + j < T; ++j) acc += conv_w[(size_t)j * D + d] * du[(size_t)(t + j) * Dh + n];
                    dx[((size_t)b * T + t) * D + d] = acc;
                    double dut = du[(size_t)t * Dh + n];
                    for (int j = 0; j < CONV_WIDTH; ++j) dconv_w[(size_t)j * D + d] += dut * x_at(x, conv_state_in, T, D, b, t - j, d);
                    if (dconv_b) dconv_b[d] += dut;
                }
            }
            /* the carried inputs x_{-3..-1}, and what arrives through the copies in conv_state_out */
            if (dconv_state_in) {
                for (int r = 0; r < CONV_WIDTH - 1; ++r)
                    for (int n = 0; n < Dh; ++n) {
                        int d = d0 + n;
                        double acc = 0.0;
                        for (int j = 0; j < CONV_WIDTH; ++j) {
                            int t = r - (CONV_WIDTH - 1) + j;
                            if (t >= 0 && t < T) acc += conv_w[(size_t)j * D + d] * du[(size_t)t * Dh + n];
                        }
                        dconv_state_in[((size_t)b * (CONV_WIDTH - 1) + r) * D + d] = acc;
                    }
            }
            if (dconv_state_out) {
                for (int k2 = 0; k2 < CONV_WIDTH - 1; ++k2)
                    for (int n = 0; n < Dh; ++n) {
                        int d = d0 + n;
                        double gk = dconv_state_out[((size_t)b * (CONV_WIDTH - 1) + k2) * D + d];
                        int row = T + k2;                       /* row of concat(conv_state_in, x) that was copied */
                        if (row >= CONV_WIDTH - 1) dx[((size_t)b * T + (row - (CONV_WIDTH - 1))) * D + d] += gk;
                        else if (dconv_state_in) dconv_state_in[((size_t)b * (CONV_WIDTH - 1) + row) * D + d] += gk;
                    }
            }
        }
        free(u);
        free(za);
        free(dzx);
    }
    return 0;
}
