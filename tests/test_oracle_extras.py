"""Pins of the oracle's optional parts: the l2 term of Section 5.1 and the
step-dependent rates of Algorithm 1 / Assumption 2, each against an independent
numpy statement of the same arithmetic."""
import numpy as np
import pytest

from _util import brute_qx

BETA, THETA, EPS, LR = 0.9, 0.999, 1e-8, 1e-3
LAMBDA = 5e-4                                               # Section 5.1


def _mk(oracle, seg_len, n, kg, kx, placement, grid=0):
    return oracle.OracleState(seg_len, n, kg, kx, placement, beta1=BETA, beta2=THETA, eps=EPS,
                              grid_g=grid)


def _adam_l2_f32(x, grads, lam, beta, theta, eps, lr):
    """Adam on the l2-regularised loss: the gradient is g + lambda x (binary32)."""
    f = np.float32
    x = np.array(x, np.float32)
    m, v = np.zeros_like(x), np.zeros_like(x)
    for g in grads:
        gg = g.astype(np.float32) + f(lam) * x
        v = f(theta) * v + (f(1) - f(theta)) * (gg * gg)
        m = f(beta) * m + (f(1) - f(beta)) * gg
        x = x - (f(lr) * m) / np.sqrt(v + f(eps))
    return x, m, v


def _adam_l2_f64(x, grads, lam, beta, theta, eps, lr):
    lam, beta, theta, eps, lr = (float(np.float32(h)) for h in (lam, beta, theta, eps, lr))
    x = np.array(x, np.float64)
    m, v = np.zeros_like(x), np.zeros_like(x)
    for g in grads:
        gg = g.astype(np.float64) + lam * x
        v = theta * v + (1 - theta) * gg * gg
        m = beta * m + (1 - beta) * gg
        x = x - lr * m / np.sqrt(v + eps)
    return x, m, v


@pytest.mark.parametrize("placement", [0, 1])
def test_l2_term_with_identity_quantizers_is_adam_on_the_regularised_loss(oracle, placement):
    rng = np.random.default_rng(3)
    d, T = 500, 20
    g = (rng.standard_normal((T, d)) * 0.01).astype(np.float32)
    x1 = (rng.standard_normal(d) * 0.3).astype(np.float32)
    st = _mk(oracle, [d], 1, -1, -1, placement)
    st.set_weights(x1)
    st.set_regularization(LAMBDA)
    for t in range(T):
        st.step(st.to_padded(g[t])[None, :], LR)
    x32, m32, v32 = _adam_l2_f32(x1, g, LAMBDA, BETA, THETA, EPS, LR)
    m = st.m if placement == oracle.PLACE_SERVER else st.m[0]
    v = st.v if placement == oracle.PLACE_SERVER else st.v[0]
    assert np.array_equal(st.to_logical(m), m32)
    assert np.array_equal(st.to_logical(v), v32)
    assert np.array_equal(st.to_logical(st.x), x32)
    x64, _, _ = _adam_l2_f64(x1, g, LAMBDA, BETA, THETA, EPS, LR)
    assert np.max(np.abs(st.to_logical(st.x) - x64)) <= 2e-6 * np.max(np.abs(x64))
    # and it is not the unregularised run
    x_plain, _, _ = _adam_l2_f32(x1, g, 0.0, BETA, THETA, EPS, LR)
    assert not np.array_equal(st.to_logical(st.x), x_plain)


@pytest.mark.parametrize("kx", [0, 1, 6])
def test_l2_term_uses_the_weights_the_workers_hold(oracle, kx):
    """With quantized weights the workers hold Q_x(x), so with a zero gradient and an
    identity Q_g what a worker sends is lambda Q_x(x) exactly (one product)."""
    rng = np.random.default_rng(kx)
    d, n = 700, 2
    x1 = (rng.standard_normal(d) * 0.3).astype(np.float32)
    st = _mk(oracle, [d], n, -1, kx, oracle.PLACE_SERVER)
    st.set_weights(x1)
    st.set_regularization(LAMBDA)
    st.workers_step(np.zeros((n, st.D), np.float32), LR)
    xhat = (brute_qx(x1, kx).astype(np.float64) / 2 ** (kx + 1)).astype(np.float32)   # exact
    want = np.float32(LAMBDA) * xhat
    for i in range(n):
        sent = st.to_logical(st.gcodes[i].view(np.float32))
        assert np.array_equal(sent, want)
    assert np.any(xhat != x1)                               # the master copy would differ


@pytest.mark.parametrize("placement", [0, 1])
@pytest.mark.parametrize("kg", [0, 1])
def test_l2_term_enters_before_quantization_and_error_feedback(oracle, placement, kg):
    """sent + e' = u with u built from g + lambda x^ (moments on the server) or from the
    moments of g + lambda x^ (moments on the workers), recomputed here in numpy."""
    f = np.float32
    rng = np.random.default_rng(10 + kg)
    seg, n, T = [300, 129], 3, 4
    d = sum(seg)
    x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
    st = _mk(oracle, seg, n, kg, 0, placement)
    st.set_weights(x1)
    st.set_regularization(LAMBDA)
    lv = oracle.grad_levels(kg, 0)
    L = len(lv) - 1
    bits = oracle.grad_code_bits(kg, 0)
    m = np.zeros((n, st.D), np.float32)
    v = np.zeros((n, st.D), np.float32)
    for t in range(T):
        g = st.to_padded((rng.standard_normal((n, d)) * 0.01).astype(np.float32))
        xhat = st.held_weights().copy()
        e_old = st.e.copy()
        st.step(g, LR)
        for i in range(n):
            gg = g[i] + f(LAMBDA) * xhat
            if placement == oracle.PLACE_WORKER:
                v[i] = f(THETA) * v[i] + (f(1) - f(THETA)) * (gg * gg)
                m[i] = f(BETA) * m[i] + (f(1) - f(BETA)) * gg
                u = (f(LR) * m[i]) / np.sqrt(v[i] + f(EPS)) + e_old[i]
            else:
                u = gg + e_old[i]
            code = oracle.unpack_bits(st.gcodes[i], st.D, bits).astype(np.int64) - L
            sent = np.zeros(st.D, np.float32)
            for s, (off, ln) in enumerate(zip(st.seg_off.tolist(), st.seg_len.tolist())):
                c = code[off:off + ln]
                mag = st.scales[i, s] * lv[np.abs(c)]
                sent[off:off + ln] = np.where(c < 0, -mag, mag)
                assert st.scales[i, s] == np.max(np.abs(u[off:off + ln]))
            assert np.array_equal(u - sent, st.e[i])


def test_step_dependent_rates_follow_a_textbook_loop(oracle):
    """Assumption 2's schedules, computed by the caller and handed over per step:
    theta_t = 1 - theta/t, alpha_t = alpha/sqrt(t), beta_t = beta * 0.9^(t-1)."""
    f = np.float32
    rng = np.random.default_rng(5)
    d, T = 400, 15
    g = (rng.standard_normal((T, d)) * 0.01).astype(np.float32)
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    st = _mk(oracle, [d], 1, -1, -1, oracle.PLACE_WORKER)
    st.set_weights(x1)
    x32 = x1.copy()
    m32, v32 = np.zeros(d, np.float32), np.zeros(d, np.float32)
    x64 = x1.astype(np.float64)
    m64, v64 = np.zeros(d), np.zeros(d)
    for t in range(1, T + 1):
        beta_t = f(0.9 * 0.9 ** (t - 1))
        theta_t = f(1.0 - 0.5 / t)
        alpha_t = f(1e-3 / np.sqrt(t))
        st.set_moment_rates(float(beta_t), float(theta_t))
        st.step(st.to_padded(g[t - 1])[None, :], float(alpha_t))
        gg = g[t - 1]
        v32 = theta_t * v32 + (f(1) - theta_t) * (gg * gg)
        m32 = beta_t * m32 + (f(1) - beta_t) * gg
        x32 = x32 - (alpha_t * m32) / np.sqrt(v32 + f(EPS))
        b, th, a = float(beta_t), float(theta_t), float(alpha_t)
        v64 = th * v64 + (1 - th) * gg.astype(np.float64) ** 2
        m64 = b * m64 + (1 - b) * gg
        x64 = x64 - a * m64 / np.sqrt(v64 + float(f(EPS)))
    assert np.array_equal(st.to_logical(st.x), x32)
    assert np.array_equal(st.to_logical(st.m[0]), m32)
    assert np.array_equal(st.to_logical(st.v[0]), v32)
    assert np.max(np.abs(st.to_logical(st.x) - x64)) <= 2e-6 * np.max(np.abs(x64))
    # theta_1 = 1/2: after one step v_1 = g^2 / 2 exactly
    st2 = _mk(oracle, [d], 1, -1, -1, oracle.PLACE_WORKER)
    st2.set_weights(x1)
    st2.set_moment_rates(0.0, 0.5)
    st2.step(st2.to_padded(g[0])[None, :], 1e-3)
    assert np.array_equal(st2.to_logical(st2.v[0]), f(0.5) * (g[0] * g[0]))
    assert np.array_equal(st2.to_logical(st2.m[0]), g[0])


# ---------------------------------------------------------------- error feedback for the broadcast

@pytest.mark.parametrize("kx", [0, 2, 6])
def test_weight_feedback_buffer_carries_the_broadcast_error(oracle, kx):
    """The optional error buffer of the broadcast (beyond the paper): what is sent is Q_x(x + e^w)
    and e^w <- (x + e^w) - Q_x(x + e^w).  Pins: each step follows that definition with Q_x from
    the rational brute force; the broadcasts telescope, sum_t Q_x(y_t) + e^w_{T+1} = sum_t x_t;
    e^w stays within half a grid step; the master weights are exactly those of a run without
    the buffer; and without the buffer nothing changes.  (Weights stay inside [-1/2, 1/2].)"""
    from _util import brute_qx
    rng = np.random.default_rng(70 + kx)
    seg, n, T = [200, 70, 130], 2, 6
    d = sum(seg)
    x1 = np.clip(rng.standard_normal(d) * 0.15, -0.4, 0.4).astype(np.float32)
    a = oracle.OracleState(seg, n, 0, kx, 0, 0.9, 0.999, 1e-8, want_wfeedback=True, want_wresid=True)
    b = oracle.OracleState(seg, n, 0, kx, 0, 0.9, 0.999, 1e-8)
    a.set_weights(x1)
    b.set_weights(x1)
    step = np.float32(2.0 ** -(kx + 1))
    sent_sum = np.zeros(a.D, np.float64)
    x_sum = np.zeros(a.D, np.float64)
    ew_before = np.zeros(a.D, np.float32)
    for t in range(T + 1):
        # the broadcast that has just been emitted is Q_x(x + e^w before it)
        y = a.x + ew_before
        q = np.zeros(a.D, np.int32)
        for off, ln in zip(a.seg_off.tolist(), a.seg_len.tolist()):
            q[off:off + ln] = brute_qx(y[off:off + ln], kx)
        xhat = q.astype(np.float32) * step
        assert np.array_equal(a.decoded_weights(), xhat)
        assert np.array_equal(a.wfeedback, y - xhat) and np.array_equal(a.wresid, a.wfeedback)
        inside = np.abs(y) <= 0.5                  # beyond the grid's end Q_x clips and the error is larger
        assert np.max(np.abs(a.wfeedback[inside])) <= 2.0 ** -(kx + 2) + 1e-12
        sent_sum += xhat
        x_sum += a.x
        assert np.array_equal(a.x, b.x), "the master copy does not depend on the buffer"
        ew_before = a.wfeedback.copy()
        if t < T:
            g = a.to_padded((rng.standard_normal((n, d)) * 0.01).astype(np.float32))
            a.step(g, 1e-2)
            b.step(g, 1e-2)
    assert np.max(np.abs(sent_sum + a.wfeedback - x_sum)) < 1e-5
    # without the buffer the broadcast is Q_x(x), and it drifts from the running mean of x further
    plain_err = np.abs(b.decoded_weights() - b.x).max()
    assert plain_err <= 2.0 ** -(kx + 2)
