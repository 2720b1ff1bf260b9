"""Pins of the CPU oracle against what the paper's equations and plain mathematics fix.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign or index, transposed
weight, reversed taps, off-by-one in the state) fails at least one of them.  None of these tests touches
the CUDA path.
"""
import math
import os

import numpy as np
import pytest

from paper_2402_19427_b200 import inputs as synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


def sigmoid(z):
    return 1.0 / (1.0 + np.exp(-z))


def identity_conv(D):
    w = np.zeros((4, D))
    w[0] = 1.0
    return w


def const_gate_params(D, H, lam, beta, gamma):
    Dh = D // H
    return dict(conv_w=identity_conv(D), conv_b=np.zeros(D), W_a=np.zeros((H, Dh, Dh)), b_a=np.full(D, beta),
                W_x=np.zeros((H, Dh, Dh)), b_x=np.full(D, gamma), lam=np.asarray(lam, dtype=np.float64))


def rand_problem(seed, B=2, T=17, D=12, H=3, scale_w=0.7):
    rng = np.random.default_rng(seed)
    Dh = D // H
    p = dict(conv_w=rng.normal(size=(4, D)) * 0.5, conv_b=rng.normal(size=D) * 0.3,
             W_a=rng.normal(size=(H, Dh, Dh)) * scale_w, b_a=rng.normal(size=D) * 0.5,
             W_x=rng.normal(size=(H, Dh, Dh)) * scale_w, b_x=rng.normal(size=D) * 0.5,
             lam=rng.uniform(-1.0, 5.0, size=D))
    x = rng.normal(size=(B, T, D))
    h0 = rng.normal(size=(B, D))
    cs = rng.normal(size=(B, 3, D))
    return x, p, h0, cs


# ---------------------------------------------------------------- P1: closed form, constant gates (Eq. 1-4)
def test_worked_example_constant_gates(oracle):
    g = read_golden("constant_gates_worked_example.txt")
    a, m = oracle.decay(0.0, 0.5, 8.0)
    assert a == g["a_t"]
    assert abs(m - g["m_t"]) < 1e-15
    T = 400
    x = np.ones((1, T, 2))
    y, hT, _ = oracle.prefill(x, const_gate_params(2, 1, [0.0, 0.0], 0.0, 0.0), H=1)
    for t in (1, 2, 3, 4):
        assert abs(y[0, t - 1, 0] - g[f"h_{t}"]) < 1e-15
    assert abs(hT[0, 1] - g["h_inf"]) < 1e-15


def test_closed_form_geometric_sum(oracle):
    rng = np.random.default_rng(1)
    D, H, T, B = 6, 2, 50, 2
    lam = rng.uniform(-2, 6, size=D)
    beta, gamma, c = 0.3, -0.4, 8.0
    x = rng.normal(size=(B, T, D))
    y, hT, _ = oracle.prefill(x, const_gate_params(D, H, lam, beta, gamma), H=H, c=c)
    alpha = sigmoid(lam) ** (c * sigmoid(beta))
    scale = np.sqrt(1 - alpha ** 2) * sigmoid(gamma)
    for t in (0, 1, 7, T - 1):
        k = np.arange(t + 1)
        ref = np.einsum("kd,bkd->bd", alpha[None, :] ** (t - k)[:, None] * scale[None, :], x[:, : t + 1])
        np.testing.assert_allclose(y[:, t], ref, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(hT, y[:, -1], rtol=0, atol=0)


# ---------------------------------------------------------------- P1b / P9 / P10: decay sign, gate curves, init
def test_decay_sign_and_lambda_init():
    import oracle
    g = read_golden("decay_sign_and_init.txt")
    a, _ = oracle.decay(2.0, 0.5, 8.0)
    assert abs(a - g["sign_a_t"]) < 1e-15
    for p in ("0.9", "0.999", "0.9999"):
        lam = float(synth.lambda_for_decay(np.array([float(p)]))[0])
        assert abs(lam - g[f"lam_p{p}"]) < 1e-9 * max(1.0, abs(lam))
        a1, m1 = oracle.decay(g[f"lam_p{p}"], 1.0, 8.0)          # alpha(1) = a^c
        assert abs(a1 - float(p)) < 1e-13
        a_unit, _ = oracle.decay(g[f"lam_p{p}"], 1.0, 1.0)       # c = 1, r = 1: a itself
        assert abs(a_unit - g[f"a_p{p}"]) < 1e-13
        assert abs(-math.log(a_unit) - g[f"softplus_neg_lam_p{p}"]) < 1e-15


def test_gate_curves(oracle):
    # alpha(r) = a^(c r), beta(r) = sqrt(1 - alpha^2) (Appendix A, gate behaviour)
    for lam in (-3.0, 0.0, 2.0, 9.0, 11.29, 30.0):
        a0, m0 = oracle.decay(lam, 0.0, 8.0)
        assert a0 == 1.0 and m0 == 0.0
        for r in (1e-6, 0.1, 0.5, 0.9, 1.0):
            a, m = oracle.decay(lam, r, 8.0)
            a_ref = math.exp(8.0 * r * math.log(1.0 / (1.0 + math.exp(-lam)))) if lam < 20 else math.exp(-8.0 * r * math.exp(-lam))
            assert abs(a - a_ref) <= 1e-12 * a_ref + 1e-300
            assert 0.0 <= a <= 1.0 and 0.0 <= m <= 1.0
            assert abs(a * a + m * m - 1.0) < 1e-12
            assert not math.isnan(m)
    # a -> 1 without cancellation: Lambda = 30, r = 1e-3: 1 - a^2 ~ 2 c r e^-30
    a, m = oracle.decay(30.0, 1e-3, 8.0)
    assert abs(m * m - 2 * 8.0 * 1e-3 * math.log1p(math.exp(-30.0))) < 1e-25


# ---------------------------------------------------------------- P2: unit stationary variance
def test_unit_stationary_variance(oracle):
    rng = np.random.default_rng(2)
    D, T = 512, 4000
    lam = synth.lambda_for_decay(np.full(D, 0.9))          # a^c = 0.9
    p = const_gate_params(D, 1, lam, 50.0, 50.0)            # r = i = 1 to ~1e-22  ->  a_t = 0.9
    x = rng.normal(size=(1, T, D))
    y, _, _ = oracle.prefill(x, p, H=1)
    tail = y[0, 500:, :]
    var = tail.var()
    n_eff = tail.size * (1 - 0.81) / (1 + 0.81)             # AR(1) effective sample size for the variance
    assert abs(var - 1.0) < 5 * math.sqrt(2.0 / n_eff)
    assert abs(tail.mean()) < 0.02


# ---------------------------------------------------------------- P3 / P4: zero input, linearity in h0
def test_zero_input_and_h0_decay(oracle):
    x, p, h0, _ = rand_problem(3)
    p["conv_b"] = np.zeros_like(p["conv_b"])
    y, hT, cs = oracle.prefill(np.zeros_like(x), p, H=3)
    assert np.all(y == 0) and np.all(hT == 0) and np.all(cs == 0)
    # zero input, h0 != 0, constant gates: h_T = sigmoid(Lambda)^(c sigmoid(b_a) T) h0
    D, T = 5, 23
    lam = np.linspace(-1, 4, D)
    pc = const_gate_params(D, 1, lam, 0.7, 0.1)
    h0 = np.arange(1, D + 1, dtype=np.float64)[None]
    _, hT, _ = oracle.prefill(np.zeros((1, T, D)), pc, H=1, h0=h0)
    np.testing.assert_allclose(hT[0], sigmoid(lam) ** (8.0 * sigmoid(0.7) * T) * h0[0], rtol=1e-12)


def test_linearity_in_h0(oracle):
    x, p, h0, cs = rand_problem(4)
    y0, _, _ = oracle.prefill(x, p, H=3, conv_state_in=cs)
    y1, _, _ = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs)
    y2, _, _ = oracle.prefill(x, p, H=3, h0=2.5 * h0, conv_state_in=cs)
    np.testing.assert_allclose(y2 - y0, 2.5 * (y1 - y0), rtol=1e-10, atol=1e-13)
    # the homogeneous part is prod_k a_k * h0 with 0 <= a_k <= 1: monotone non-increasing magnitude
    ratio = np.abs(y1 - y0) / np.abs(h0)[:, None, :]
    assert np.all(np.diff(ratio, axis=1) <= 1e-12) and np.all(ratio <= 1.0 + 1e-12)


# ---------------------------------------------------------------- P5: prefill == chained decode == split prefill
def test_prefill_equals_chained_decode_and_split(oracle):
    x, p, h0, cs = rand_problem(5, T=19)
    B, T, D = x.shape
    y, hT, cso = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs)
    h, c = h0.copy(), cs.copy()
    for t in range(T):
        yt, h, c = oracle.decode_step(x[:, t], p, 3, h, c)
        np.testing.assert_allclose(yt, y[:, t], rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(h, hT, rtol=1e-13, atol=1e-14)
    assert np.array_equal(c, cso)
    assert np.array_equal(cso, x[:, -3:])                       # raw inputs, oldest first
    for T1 in (1, 2, 3, 7):
        ya, ha, ca = oracle.prefill(x[:, :T1], p, H=3, h0=h0, conv_state_in=cs)
        yb, hb, cb = oracle.prefill(x[:, T1:], p, H=3, h0=ha, conv_state_in=ca)
        np.testing.assert_allclose(np.concatenate([ya, yb], 1), y, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(hb, hT, rtol=1e-13, atol=1e-14)
        assert np.array_equal(cb, cso)
        # T < 3 keeps the tail of the old state
        expect = np.concatenate([cs, x[:, :T1]], 1)[:, -3:]
        assert np.array_equal(ca, expect)


# ---------------------------------------------------------------- P7: structural invariants
def test_causality_head_and_batch_independence(oracle):
    x, p, h0, cs = rand_problem(6, B=3, T=15, D=12, H=3)
    y, _, _ = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs)
    x2 = x.copy()
    x2[:, 9:] += 1.0                                            # future change
    y2, _, _ = oracle.prefill(x2, p, H=3, h0=h0, conv_state_in=cs)
    assert np.array_equal(y2[:, :9], y[:, :9]) and not np.array_equal(y2[:, 9], y[:, 9])
    x3 = x.copy()
    x3[:, :, 4:8] += 1.0                                        # head 1 only
    y3, _, _ = oracle.prefill(x3, p, H=3, h0=h0, conv_state_in=cs)
    assert np.array_equal(y3[:, :, :4], y[:, :, :4]) and np.array_equal(y3[:, :, 8:], y[:, :, 8:])
    assert np.all(y3[:, 3:, 4:8] != y[:, 3:, 4:8])              # every channel of the head sees it (dense block)
    x4 = x.copy()
    x4[1] += 1.0                                                # batch row 1 only
    y4, _, _ = oracle.prefill(x4, p, H=3, h0=h0, conv_state_in=cs)
    assert np.array_equal(y4[0], y[0]) and np.array_equal(y4[2], y[2])
    # head slicing is self-contained
    inp = dict(B=3, T=15, D=12, H=3, x=x, params=p, h0=h0, conv_state=cs)
    s = synth.head_slice(inp, [2], batches=[1])
    ys, _, _ = oracle.prefill(s["x"], s["params"], H=1, h0=s["h0"], conv_state_in=s["conv_state"])
    assert np.array_equal(ys[0], y[1, :, 8:])


# ---------------------------------------------------------------- P8: rebuild from textbook/library routines
def independent_forward(x, p, H, h0, cs, c=8.0, chunk=5):
    """Third implementation from library routines only: torch conv1d (left pad 3), batched matmul + logistic,
    and a chunked fold of the monoid (a2 a1, a2 b1 + b2).  Shares no code with the oracle."""
    import torch
    B, T, D = x.shape
    Dh = D // H
    xt = torch.from_numpy(np.concatenate([cs, x], axis=1)).permute(0, 2, 1)          # [B, D, T+3]
    w = torch.from_numpy(p["conv_w"][::-1].copy()).permute(1, 0).unsqueeze(1)        # [D,1,4]: kernel[k] hits x_{t-3+k}
    u = torch.nn.functional.conv1d(xt, w, bias=torch.from_numpy(p["conv_b"]), groups=D).permute(0, 2, 1).numpy()
    uh = u.reshape(B, T, H, Dh)
    za = np.einsum("hon,bthn->btho", p["W_a"], uh).reshape(B, T, D) + p["b_a"]
    zx = np.einsum("hon,bthn->btho", p["W_x"], uh).reshape(B, T, D) + p["b_x"]
    r, i = sigmoid(za), sigmoid(zx)
    a = sigmoid(p["lam"]) ** (c * r)
    bterm = np.sqrt(1 - a ** 2) * i * u
    # chunked association: fold each chunk to (A, Bc), then combine chunk aggregates left to right
    y = np.empty_like(x)
    h = h0.copy()
    for s in range(0, T, chunk):
        A = np.ones((B, D)); Bc = np.zeros((B, D))
        local = []
        for t in range(s, min(T, s + chunk)):
            A, Bc = a[:, t] * A, a[:, t] * Bc + bterm[:, t]
            local.append((A.copy(), Bc.copy()))
        for k, (Ak, Bk) in enumerate(local):
            y[:, s + k] = Ak * h + Bk
        h = A * h + Bc
    return y, h


def test_against_library_reconstruction(oracle):
    x, p, h0, cs = rand_problem(7, B=2, T=23, D=12, H=3)
    p["lam"] = np.random.default_rng(70).uniform(-1.0, 6.0, size=12)
    y, hT, _ = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs)
    yr, hr = independent_forward(x, p, 3, h0, cs)
    np.testing.assert_allclose(y, yr, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(hT, hr, rtol=1e-11, atol=1e-12)
    # non-default c
    y5, _, _ = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs, c=5.0)
    yr5, _ = independent_forward(x, p, 3, h0, cs, c=5.0)
    np.testing.assert_allclose(y5, yr5, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------- P6: backward vs central finite differences
def loss(oracle, x, p, H, dy, h0, cs):
    y, _, _ = oracle.prefill(x, p, H=H, h0=h0, conv_state_in=cs)
    return float(np.sum(dy * y))


@pytest.mark.parametrize("shape", [dict(B=2, T=64, D=64, H=2), dict(B=1, T=5, D=6, H=3)])
def test_backward_central_differences(oracle, shape):
    rng = np.random.default_rng(8)
    B, T, D, H = shape["B"], shape["T"], shape["D"], shape["H"]
    x, p, h0, cs = rand_problem(9, B=B, T=T, D=D, H=H, scale_w=1.0 / math.sqrt(D // H))
    p["lam"] = rng.uniform(0.5, 5.0, size=D)
    dy = rng.normal(size=(B, T, D))
    g = oracle.backward(x, p, H, dy, h0=h0, conv_state_in=cs)
    eps = 1e-6

    def fd(get, put, idx):
        old = get()[idx]
        put(idx, old + eps); lp = loss(oracle, x, p, H, dy, h0, cs)
        put(idx, old - eps); lm = loss(oracle, x, p, H, dy, h0, cs)
        put(idx, old)
        return (lp - lm) / (2 * eps)

    def check(name, arr, grad, n=6):
        flat_idx = rng.choice(arr.size, size=min(n, arr.size), replace=False)
        scale = np.abs(grad).max() + 1e-30
        for fi in flat_idx:
            idx = np.unravel_index(fi, arr.shape)
            num = fd(lambda: arr, lambda i, v: arr.__setitem__(i, v), idx)
            assert abs(num - grad[idx]) <= 2e-6 * scale + 1e-7 * abs(num), (name, idx, num, grad[idx])

    check("x", x, g["x"], n=10)
    for name in ("conv_w", "conv_b", "W_a", "b_a", "W_x", "b_x", "lam"):
        check(name, p[name], g[name])
    # the earliest tokens and the last token (edges of the anti-causal conv and of the reverse scan)
    for idx in [(0, 0, 0), (0, T - 1, D - 1), (B - 1, 1, 1), (B - 1, T - 2, 2)]:
        num = fd(lambda: x, lambda i, v: x.__setitem__(i, v), idx)
        assert abs(num - g["x"][idx]) <= 2e-6 * (np.abs(g["x"]).max()) + 1e-7 * abs(num)


def test_backward_directional_derivative(oracle):
    # <grad, delta> == d/d eps loss(theta + eps delta) for a random direction over all inputs at once
    rng = np.random.default_rng(10)
    B, T, D, H = 2, 24, 16, 2
    x, p, h0, cs = rand_problem(11, B=B, T=T, D=D, H=H)
    dy = rng.normal(size=(B, T, D))
    g = oracle.backward(x, p, H, dy, h0=h0, conv_state_in=cs)
    dirs = {k: rng.normal(size=v.shape) for k, v in p.items()}
    dx = rng.normal(size=x.shape)
    eps = 1e-6

    def shifted(s):
        return x + s * dx, {k: v + s * dirs[k] for k, v in p.items()}

    xp, pp = shifted(eps); xm, pm = shifted(-eps)
    num = (loss(oracle, xp, pp, H, dy, h0, cs) - loss(oracle, xm, pm, H, dy, h0, cs)) / (2 * eps)
    ana = float(np.sum(g["x"] * dx) + sum(np.sum(g[k] * dirs[k]) for k in p))
    assert abs(num - ana) <= 1e-6 * max(1.0, abs(ana))


def test_backward_overwrites_and_is_additive_in_batch(oracle):
    # parameter gradients sum over the batch; dx rows are per-sequence
    rng = np.random.default_rng(12)
    x, p, h0, cs = rand_problem(13, B=3, T=9, D=8, H=2)
    dy = rng.normal(size=x.shape)
    g = oracle.backward(x, p, 2, dy, h0=h0, conv_state_in=cs)
    parts = [oracle.backward(x[b:b + 1], p, 2, dy[b:b + 1], h0=h0[b:b + 1], conv_state_in=cs[b:b + 1]) for b in range(3)]
    for k in p:
        np.testing.assert_allclose(g[k], sum(q[k] for q in parts), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(g["x"], np.concatenate([q["x"] for q in parts], 0), rtol=0, atol=0)


def loss_with_state(oracle, x, p, H, dy, h0, cs, dhT, dcs):
    y, hT, cso = oracle.prefill(x, p, H=H, h0=h0, conv_state_in=cs)
    return float(np.sum(dy * y) + np.sum(dhT * hT) + np.sum(dcs * cso))


@pytest.mark.parametrize("shape", [dict(B=2, T=33, D=16, H=2), dict(B=1, T=2, D=6, H=3), dict(B=2, T=1, D=4, H=1)])
def test_backward_state_gradients_central_differences(oracle, shape):
    """dh0 and d conv_state_in, with gradient arriving through h_T and conv_state_out as well (the terms a later segment of
    the sequence sends back): central differences of loss = <dy,y> + <dh_T,h_T> + <dcs_out,cs_out> in fp64.  T = 1, 2: the
    conv state is partly a copy of the incoming one, so part of dcs_out passes straight through."""
    rng = np.random.default_rng(21)
    B, T, D, H = shape["B"], shape["T"], shape["D"], shape["H"]
    x, p, h0, cs = rand_problem(22, B=B, T=T, D=D, H=H, scale_w=1.0 / math.sqrt(D // H))
    p["lam"] = rng.uniform(0.5, 5.0, size=D)
    dy = rng.normal(size=(B, T, D)); dhT = rng.normal(size=(B, D)); dcs = rng.normal(size=(B, 3, D))
    g = oracle.backward(x, p, H, dy, h0=h0, conv_state_in=cs, dh_T=dhT, dconv_state_out=dcs, state_grads=True)
    eps = 1e-6

    def fd(arr, idx):
        old = arr[idx]
        arr[idx] = old + eps; lp = loss_with_state(oracle, x, p, H, dy, h0, cs, dhT, dcs)
        arr[idx] = old - eps; lm = loss_with_state(oracle, x, p, H, dy, h0, cs, dhT, dcs)
        arr[idx] = old
        return (lp - lm) / (2 * eps)

    for name, arr, grad in (("h0", h0, g["h0"]), ("conv_state", cs, g["conv_state"]), ("x", x, g["x"]), ("lam", p["lam"], g["lam"]),
                            ("conv_w", p["conv_w"], g["conv_w"]), ("W_a", p["W_a"], g["W_a"])):
        scale = np.abs(grad).max() + 1e-30
        for fi in rng.choice(arr.size, size=min(8, arr.size), replace=False):
            idx = np.unravel_index(fi, arr.shape)
            num = fd(arr, idx)
            assert abs(num - grad[idx]) <= 2e-6 * scale + 1e-7 * abs(num), (name, idx, num, grad[idx])
    # every row of the carried conv inputs, first and last channel
    for idx in [(0, 0, 0), (0, 1, D - 1), (B - 1, 2, 0)]:
        assert abs(fd(cs, idx) - g["conv_state"][idx]) <= 2e-6 * (np.abs(g["conv_state"]).max() + 1e-30)


def test_backward_without_incoming_state_gradient_is_unchanged_and_dh0_is_the_decay_product(oracle):
    rng = np.random.default_rng(23)
    x, p, h0, cs = rand_problem(24, B=2, T=12, D=8, H=2)
    dy = rng.normal(size=x.shape)
    g0 = oracle.backward(x, p, 2, dy, h0=h0, conv_state_in=cs)
    g1 = oracle.backward(x, p, 2, dy, h0=h0, conv_state_in=cs, state_grads=True)
    for k in g0:
        assert np.array_equal(g0[k], g1[k])
    # gates do not see h (Eq. 1-3), so y_t depends on h0 only through prod_{k<=t} a_k: dh0 = sum_t dy_t prod_{k<=t} a_k
    y1, _, _ = oracle.prefill(x, p, H=2, h0=h0 + 1.0, conv_state_in=cs)
    y0, _, _ = oracle.prefill(x, p, H=2, h0=h0, conv_state_in=cs)
    np.testing.assert_allclose(g1["h0"], np.sum(dy * (y1 - y0), axis=1), rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("T1,T2", [(7, 9), (1, 5), (2, 2), (6, 1)])
def test_backward_of_two_chained_segments_equals_one_segment(oracle, T1, T2):
    """Truncated segments compose: the second segment's dh0 and d conv_state_in are the first segment's dh_T and
    d conv_state_out; dx concatenates, parameter gradients add, and the first segment's state gradients are the whole's."""
    rng = np.random.default_rng(25)
    B, D, H = 2, 8, 2
    x, p, h0, cs = rand_problem(26, B=B, T=T1 + T2, D=D, H=H)
    dy = rng.normal(size=x.shape); dhT = rng.normal(size=(B, D)); dcs = rng.normal(size=(B, 3, D))
    whole = oracle.backward(x, p, H, dy, h0=h0, conv_state_in=cs, dh_T=dhT, dconv_state_out=dcs, state_grads=True)
    _, h1, cs1 = oracle.prefill(x[:, :T1], p, H=H, h0=h0, conv_state_in=cs)
    g2 = oracle.backward(x[:, T1:], p, H, dy[:, T1:], h0=h1, conv_state_in=cs1, dh_T=dhT, dconv_state_out=dcs, state_grads=True)
    g1 = oracle.backward(x[:, :T1], p, H, dy[:, :T1], h0=h0, conv_state_in=cs, dh_T=g2["h0"], dconv_state_out=g2["conv_state"],
                         state_grads=True)
    np.testing.assert_allclose(np.concatenate([g1["x"], g2["x"]], 1), whole["x"], rtol=1e-10, atol=1e-12)
    for k in p:
        np.testing.assert_allclose(g1[k] + g2[k], whole[k], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g1["h0"], whole["h0"], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g1["conv_state"], whole["conv_state"], rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------- the call as one affine step, and the merged output
def test_decay_product_describes_the_call_as_one_step(oracle):
    """Eq. 4 is affine in the incoming state: h_T(h0) = (prod_t a_t) h0 + h_T(0).  The product must reproduce that for any
    h0, equal the closed form for constant gates, and compose over a split in time like the monoid (a2 a1, a2 b1 + b2)."""
    x, p, h0, cs = rand_problem(31, T=17)
    _, hz, _, ap = oracle.prefill(x, p, H=3, conv_state_in=cs, with_a_prod=True)
    _, h1, _, ap1 = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs, with_a_prod=True)
    assert np.array_equal(ap, ap1)                                  # the product does not depend on the state
    assert np.all(ap > 0) and np.all(ap < 1)
    np.testing.assert_allclose(h1, ap * h0 + hz, rtol=1e-12, atol=1e-14)
    # constant gates: a_t = sigmoid(Lambda)^(c sigmoid(b_a)) for every t
    D, T = 5, 23
    lam = np.linspace(-1, 4, D)
    pc = const_gate_params(D, 1, lam, 0.7, 0.1)
    rng = np.random.default_rng(2)
    _, _, _, apc = oracle.prefill(rng.standard_normal((2, T, D)), pc, H=1, with_a_prod=True)
    np.testing.assert_allclose(apc, np.broadcast_to(sigmoid(lam) ** (8.0 * sigmoid(0.7) * T), (2, D)), rtol=1e-12)
    # two segments: the halo of the second is the conv state of the first; aggregates combine as (a2 a1, a2 b1 + b2)
    for T1 in (1, 3, 9):
        _, b1, c1, a1 = oracle.prefill(x[:, :T1], p, H=3, conv_state_in=cs, with_a_prod=True)
        _, b2, _, a2 = oracle.prefill(x[:, T1:], p, H=3, conv_state_in=c1, with_a_prod=True)
        np.testing.assert_allclose(a2 * a1, ap, rtol=1e-12)
        np.testing.assert_allclose(a2 * b1 + b2, hz, rtol=1e-12, atol=1e-14)


def test_gelu_merge(oracle):
    """Section 2.3: GeLU on the second branch, then element-wise multiplication.  GeLU(v) = v Phi(v): GeLU(0) = 0,
    GeLU(v) - GeLU(-v) = v, GeLU(v) -> v for large v, its minimum is about -0.17 near v = -0.75, and Phi is the normal
    distribution function (checked against a numerical integral of the density).  The state is not touched by the merge."""
    assert oracle.gelu(0.0) == 0.0
    for v in (0.1, 0.5, 1.0, 2.5, 7.0):
        assert abs(oracle.gelu(v) - oracle.gelu(-v) - v) < 1e-15 * max(1.0, v)
    assert abs(oracle.gelu(12.0) - 12.0) < 1e-15 and abs(oracle.gelu(-12.0)) < 1e-15
    grid = np.linspace(-3, 0, 3001)
    vals = np.array([oracle.gelu(v) for v in grid])
    assert abs(vals.min() - (-0.16997)) < 1e-4 and abs(grid[vals.argmin()] - (-0.7518)) < 2e-3
    for v in (-1.3, 0.4, 2.0):   # Phi(v) by Simpson's rule on the normal density
        t = np.linspace(-12.0, v, 200001)
        dens = np.exp(-0.5 * t * t) / math.sqrt(2 * math.pi)
        hstep = t[1] - t[0]
        phi = hstep / 3 * (dens[0] + dens[-1] + 4 * dens[1:-1:2].sum() + 2 * dens[2:-1:2].sum())
        assert abs(oracle.gelu(v) - v * phi) < 1e-10
    x, p, h0, cs = rand_problem(32, T=11)
    rng = np.random.default_rng(5)
    g = rng.standard_normal(x.shape) * 2
    y, hT, cso = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs)
    ym, hTm, csm = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs, gate_branch=g)
    assert np.array_equal(hT, hTm) and np.array_equal(cso, csm)
    gel = np.vectorize(oracle.gelu)(g)
    np.testing.assert_allclose(ym, y * gel, rtol=1e-15, atol=0)
    # a branch that is a large constant passes h through scaled by that constant; a zero branch gives zero
    yb, _, _ = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs, gate_branch=np.full(x.shape, 20.0))
    np.testing.assert_allclose(yb, 20.0 * y, rtol=1e-14)
    y0, _, _ = oracle.prefill(x, p, H=3, h0=h0, conv_state_in=cs, gate_branch=np.zeros(x.shape))
    assert np.all(y0 == 0)


# ---------------------------------------------------------------- the synthetic input recipe
def test_input_generator_is_seeded_and_bf16_exact():
    a = synth.make_inputs(2, 16, 32, 2, io="bf16", seed=5, long_memory_frac=0.25, with_dy=True, with_state=True)
    b = synth.make_inputs(2, 16, 32, 2, io="bf16", seed=5, long_memory_frac=0.25, with_dy=True, with_state=True)
    assert np.array_equal(a["x"], b["x"]) and np.array_equal(a["params"]["W_a"], b["params"]["W_a"])
    for arr in (a["x"], a["dy"], a["conv_state"], a["params"]["conv_w"], a["params"]["W_a"], a["params"]["W_x"]):
        bits = synth.bf16_bits(arr)                                   # raises if not representable
        assert np.array_equal(synth.from_bf16_bits(bits), arr)
    apc = (1 / (1 + np.exp(-a["params"]["lam"].astype(np.float64)))) ** 8
    assert np.sum(np.abs(apc - 0.9999) < 2e-6) == 8                   # 25 % of 32 channels forced to long memory
    rest = apc[np.abs(apc - 0.9999) >= 2e-6]
    assert rest.min() >= 0.9 - 1e-5 and rest.max() <= 0.999 + 1e-5
    # RNE rounding of bf16: 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 is a tie -> 1 + 2^-6
    t = synth.round_to_bf16(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20], np.float32))
    assert t[0] == 1.0 and t[1] == np.float32(1 + 2.0 ** -6) and t[2] == np.float32(1 + 2.0 ** -7)
    for cid, cfg in synth.CONFIGS.items():
        assert cfg["D"] % cfg["H"] == 0
