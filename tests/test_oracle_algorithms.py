"""Pins of the oracle's step functions (Algorithms 1-3) against independent
statements: a textbook generic-Adam loop, the error-feedback recursion
recomputed from what was sent, the telescoping sum, the virtual iterate of the
proofs, and hand-checkable special cases."""
import numpy as np
import pytest

from _util import generic_adam_f32, generic_adam_f64

BETA, THETA, EPS, LR = 0.9, 0.999, 1e-8, 1e-3
PAPER_HYPER = dict(beta1=0.99, beta2=0.999, eps=1e-5)       # Section 5.1


def _mk(oracle, seg_len, n, kg, kx, placement, grid=0, hyper=None, wresid=False):
    h = dict(beta1=BETA, beta2=THETA, eps=EPS)
    if hyper:
        h.update(hyper)
    return oracle.OracleState(seg_len, n, kg, kx, placement, grid_g=grid, want_wresid=wresid, **h)


def _grads(rng, T, n, d, sigma=0.01):
    return (rng.standard_normal((T, n, d)) * sigma).astype(np.float32)


def _decode_stream(oracle, st, i):
    """Values worker i sent, recomputed in numpy from codes and scales."""
    lv = oracle.grad_levels(st.kg, st.grid_g)
    L = len(lv) - 1
    bits = oracle.grad_code_bits(st.kg, st.grid_g)
    code = oracle.unpack_bits(st.gcodes[i], st.D, bits).astype(np.int64) - L
    out = np.zeros(st.D, np.float32)
    for s, (off, ln) in enumerate(zip(st.seg_off.tolist(), st.seg_len.tolist())):
        c = code[off:off + ln]
        mag = st.scales[i, s] * lv[np.abs(c)]                   # fl(scale * level)
        out[off:off + ln] = np.where(c < 0, -mag, mag) * (c != 0)
        # pads must carry level 0
        pad = code[off + ln: off + (ln + 127) // 128 * 128]
        assert not pad.any()
    return out


# ---------------------------------------------------------------- layout

def test_padded_layout(oracle):
    off, D = oracle.layout([64, 129, 128, 1, 1000])
    assert off.tolist() == [0, 128, 384, 512, 640]
    assert D == 640 + 1024
    st = _mk(oracle, [64, 129, 5], 2, 0, 0, oracle.PLACE_SERVER)
    lg = np.arange(198, dtype=np.float32)
    pd = st.to_padded(lg)
    assert pd.shape == (st.D,) and pd.sum() == lg.sum()
    assert np.array_equal(st.to_logical(pd), lg)
    assert st.gcode_bytes == st.D * 2 // 8 and st.wcode_bytes == st.D * 2 // 8


# ---------------------------------------------------------------- reduction to Adam

def test_single_machine_identity_is_generic_adam(oracle):
    # Algorithm 1 with Q_g = Q_x = identity (N = 1, moments on the worker)
    rng = np.random.default_rng(0)
    d, T = 777, 25
    g = _grads(rng, T, 1, d)
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    st = _mk(oracle, [d], 1, -1, -1, oracle.PLACE_WORKER)
    st.set_weights(x1)
    for t in range(T):
        st.step(st.to_padded(g[t]), LR)
    x32, m32, v32 = generic_adam_f32(x1, g[:, 0], BETA, THETA, EPS, LR)
    # same operations, same order -> same bits, except the split x - (0 + step)
    assert np.array_equal(st.to_logical(st.m[0]), m32)
    assert np.array_equal(st.to_logical(st.v[0]), v32)
    assert np.array_equal(st.to_logical(st.x), x32)
    assert not st.e.any()
    x64, m64, v64 = generic_adam_f64(x1, g[:, 0], BETA, THETA, EPS, LR)
    assert np.max(np.abs(st.to_logical(st.x) - x64)) <= 1e-6 * np.max(np.abs(x64))


@pytest.mark.parametrize("n", [2, 4, 8])
def test_server_placement_identity_is_adam_on_mean_gradient(oracle, n):
    rng = np.random.default_rng(n)
    d, T = 300, 12
    g = _grads(rng, T, n, d)
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    st = _mk(oracle, [d], n, -1, -1, oracle.PLACE_SERVER)
    st.set_weights(x1)
    for t in range(T):
        st.step(st.to_padded(g[t]), LR)
    gbar = np.zeros((T, d), np.float32)
    for t in range(T):
        acc = np.zeros(d, np.float32)
        for i in range(n):
            acc = acc + g[t, i]
        gbar[t] = acc / np.float32(n)
    x32, m32, v32 = generic_adam_f32(x1, gbar, BETA, THETA, EPS, LR)
    assert np.array_equal(st.to_logical(st.x), x32)
    assert np.array_equal(st.to_logical(st.m), m32)
    assert np.array_equal(st.to_logical(st.v), v32)
    x64, _, _ = generic_adam_f64(x1, g.astype(np.float64).mean(axis=1), BETA, THETA, EPS, LR)
    assert np.max(np.abs(st.to_logical(st.x) - x64)) <= 2e-6 * np.max(np.abs(x64))


def test_worker_placement_identity_is_mean_of_local_adam_steps(oracle):
    # Algorithms 2-3 with identity quantizers: distributed Adam with N local rates
    rng = np.random.default_rng(7)
    n, d, T = 3, 200, 10
    g = _grads(rng, T, n, d)
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    st = _mk(oracle, [d], n, -1, -1, oracle.PLACE_WORKER, hyper=PAPER_HYPER)
    st.set_weights(x1)
    for t in range(T):
        st.step(st.to_padded(g[t]), LR)
    b, th, eps = (float(np.float32(PAPER_HYPER[k])) for k in ("beta1", "beta2", "eps"))
    lr = float(np.float32(LR))
    x = x1.astype(np.float64)
    m = np.zeros((n, d))
    v = np.zeros((n, d))
    for t in range(T):
        v = th * v + (1 - th) * g[t].astype(np.float64) ** 2
        m = b * m + (1 - b) * g[t]
        x = x - (lr * m / np.sqrt(v + eps)).mean(axis=0)
    assert np.max(np.abs(st.to_logical(st.x) - x)) <= 2e-6 * np.max(np.abs(x))
    assert np.max(np.abs(st.to_logical(st.m) - m)) <= 2e-6 * np.max(np.abs(m))
    assert np.max(np.abs(st.to_logical(st.v) - v)) <= 2e-6 * np.max(np.abs(v))


# ---------------------------------------------------------------- error feedback

@pytest.mark.parametrize("placement", [0, 1])
@pytest.mark.parametrize("kg,grid", [(0, 0), (1, 0), (2, 0), (2, 1)])
def test_error_feedback_recursion_from_what_was_sent(oracle, placement, kg, grid):
    """e_{t+1} = (input_t + e_t) - Q_g(input_t + e_t), with Q_g(.) rebuilt from the
    packed codes and scales exactly as a receiver would."""
    rng = np.random.default_rng(31 * kg + placement)
    seg = [130, 64, 1000, 7]
    n, T = 3, 6
    d = sum(seg)
    st = _mk(oracle, seg, n, kg, 0, placement, grid=grid)
    st.set_weights((rng.standard_normal(d) * 0.05).astype(np.float32))
    g = _grads(rng, T, n, d)
    # an independent copy of the moments for the worker placement
    f = np.float32
    m = np.zeros((n, st.D), np.float32)
    v = np.zeros((n, st.D), np.float32)
    for t in range(T):
        gp = st.to_padded(g[t])
        e_before = st.e.copy()
        st.workers_step(gp, LR)
        for i in range(n):
            if placement == oracle.PLACE_WORKER:
                v[i] = f(THETA) * v[i] + (f(1) - f(THETA)) * (gp[i] * gp[i])
                m[i] = f(BETA) * m[i] + (f(1) - f(BETA)) * gp[i]
                u = (f(LR) * m[i]) / np.sqrt(v[i] + f(EPS)) + e_before[i]
            else:
                u = gp[i] + e_before[i]
            sent = _decode_stream(oracle, st, i)
            assert np.array_equal(st.e[i], u - sent)
            # scale is the max-abs of what was quantized, per segment
            for s, (off, ln) in enumerate(zip(st.seg_off.tolist(), st.seg_len.tolist())):
                assert st.scales[i, s] == np.max(np.abs(u[off:off + ln]))
        st.server_step(LR)


def test_error_feedback_telescopes(oracle):
    # sum_t Q_g(u_t) + e_{T+1} = sum_t g_t  (server placement, input = g)
    rng = np.random.default_rng(2)
    d, T = 2000, 40
    st = _mk(oracle, [d], 1, 0, -1, oracle.PLACE_SERVER)
    g = _grads(rng, T, 1, d)
    sent_sum = np.zeros(st.D, np.float64)
    for t in range(T):
        st.workers_step(st.to_padded(g[t]), LR)
        sent_sum += _decode_stream(oracle, st, 0)
    total = g[:, 0].astype(np.float64).sum(axis=0)
    lhs = st.to_logical(sent_sum + st.e[0])
    assert np.max(np.abs(lhs - total)) <= 1e-6 * np.max(np.abs(g)) * T


def test_error_norm_is_bounded_by_the_lemma(oracle):
    """|e_{t+1}| <= sum_i (1-delta_g)^{t-i+1} |Delta_i| needs a contraction factor;
    per step it gives |e_{t+1}| <= (1-delta_g)(|in_t| + |e_t|) < |in_t| + |e_t|."""
    rng = np.random.default_rng(9)
    d, T = 512, 30
    st = _mk(oracle, [d], 1, 0, -1, oracle.PLACE_SERVER)
    g = _grads(rng, T, 1, d)
    for t in range(T):
        e0 = np.linalg.norm(st.e[0].astype(np.float64))
        st.workers_step(st.to_padded(g[t]), LR)
        e1 = np.linalg.norm(st.e[0].astype(np.float64))
        assert e1 < np.linalg.norm(g[t, 0].astype(np.float64)) + e0


# ---------------------------------------------------------------- virtual iterate

@pytest.mark.parametrize("kg", [0, 1])
def test_virtual_iterate_is_quantizer_independent(oracle, kg):
    """x~_t = x_t - (1/N) sum_i e_t^(i) obeys x~_{t+1} = x~_t + (1/N) sum_i Delta_t^(i)
    whatever Q_g is (notation of the multi-worker proof).  With gradients that do
    not depend on x, the local steps Delta are the same for every Q_g, so the
    quantized run's virtual iterate equals the unquantized run's x."""
    rng = np.random.default_rng(12)
    n, d, T = 4, 600, 30
    g = _grads(rng, T, n, d)
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    runs = {}
    for k in (-1, kg):
        st = _mk(oracle, [d], n, k, -1, oracle.PLACE_WORKER, hyper=PAPER_HYPER)
        st.set_weights(x1)
        for t in range(T):
            st.step(st.to_padded(g[t]), LR)
        runs[k] = st
    ref = runs[-1].x.astype(np.float64)
    q = runs[kg]
    virt = q.x.astype(np.float64) - q.e.astype(np.float64).mean(axis=0)
    assert np.max(np.abs(virt - ref)) <= 1e-5 * np.max(np.abs(ref))
    # and the quantized run really did quantize (so the check is not vacuous)
    assert np.max(np.abs(q.x - runs[-1].x)) > 1e-6
    # moments do not depend on the quantizer at all
    assert np.array_equal(q.m, runs[-1].m) and np.array_equal(q.v, runs[-1].v)


# ---------------------------------------------------------------- server details

def test_server_average_order_scale_and_sign(oracle):
    """A case small enough to do by hand: two workers, ternary codes."""
    st = _mk(oracle, [4], 2, 0, -1, oracle.PLACE_WORKER)
    st.set_weights(np.array([1.0, 1.0, 1.0, 1.0], np.float32))
    # craft what the workers sent: worker 0 scale 2: [+,0,-,+]; worker 1 scale 6: [-,-,0,+]
    codes0 = np.full(st.D, 1, np.uint32); codes0[:4] = [2, 1, 0, 2]
    codes1 = np.full(st.D, 1, np.uint32); codes1[:4] = [0, 0, 1, 2]
    st.gcodes[0] = oracle.pack_bits(codes0, 2)
    st.gcodes[1] = oracle.pack_bits(codes1, 2)
    st.scales[:] = [[2.0], [6.0]]
    st.server_step(LR)
    # delta^ = ([2,0,-2,2] + [-6,-6,0,6]) / 2 = [-2,-3,-1,4];  x <- x - delta^
    assert st.x[:4].tolist() == [3.0, 4.0, 2.0, -3.0]
    assert not st.x[4:].any()


def test_server_placement_step_matches_numpy(oracle):
    rng = np.random.default_rng(4)
    seg, n = [300, 77], 5
    st = _mk(oracle, seg, n, 1, 2, oracle.PLACE_SERVER, wresid=True)
    d = sum(seg)
    st.set_weights((rng.standard_normal(d) * 0.2).astype(np.float32))
    g = _grads(rng, 3, n, d)
    f = np.float32
    for t in range(3):
        st.workers_step(st.to_padded(g[t]), LR)
        x0, m0, v0 = st.x.copy(), st.m.copy(), st.v.copy()
        acc = np.zeros(st.D, np.float32)
        for i in range(n):
            acc = acc + _decode_stream(oracle, st, i)
        dhat = acc / f(n)
        v1 = f(THETA) * v0 + (f(1) - f(THETA)) * (dhat * dhat)
        m1 = f(BETA) * m0 + (f(1) - f(BETA)) * dhat
        x1 = x0 - (f(LR) * m1) / np.sqrt(v1 + f(EPS))
        st.server_step(LR)
        assert np.array_equal(st.v, v1) and np.array_equal(st.m, m1) and np.array_equal(st.x, x1)
        # broadcast = Q_x of the new master copy; residual recovers it
        xh = st.decoded_weights()
        q, xh2, r = oracle.quantize_weights(st.x, 2)
        assert np.array_equal(st.to_logical(xh), st.to_logical(xh2))
        assert np.array_equal(st.to_logical(st.wresid), st.to_logical(r))
        inside = np.abs(st.x) <= 0.5
        assert np.array_equal((xh + st.wresid)[inside], st.x[inside])


def test_first_broadcast_is_qx_of_x1(oracle):
    rng = np.random.default_rng(8)
    st = _mk(oracle, [500], 2, 0, 1, oracle.PLACE_WORKER)
    x1 = (rng.standard_normal(500) * 0.3).astype(np.float32)
    st.set_weights(x1)
    q, xh, _ = oracle.quantize_weights(x1, 1)
    assert np.array_equal(st.to_logical(st.decoded_weights()), xh)


def test_threads_only_run_workers_side_by_side(oracle):
    rng = np.random.default_rng(5)
    seg, n = [1000, 333], 6
    g = _grads(rng, 2, n, sum(seg))
    a = _mk(oracle, seg, n, 0, 0, oracle.PLACE_WORKER)
    b = _mk(oracle, seg, n, 0, 0, oracle.PLACE_WORKER)
    for t in range(2):
        a.step(a.to_padded(g[t]), LR, threads=1)
        b.step(b.to_padded(g[t]), LR, threads=4)
    for name in ("x", "m", "v", "e", "scales", "gcodes", "wcodes"):
        assert np.array_equal(getattr(a, name), getattr(b, name))
