"""CUDA library vs CPU oracle, element by element, through the C interface.

Packed codes, scales and packed weights must be byte-identical.  The fp32 state
(x, m, v, e) must agree to a maximum relative error of 1e-5 (the stated bound);
because both sides perform the same IEEE-754 binary32 operations in the same
order it is in fact required to be bit-identical here, which is what keeps the
codes identical over many steps."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from _parity import Pair, bits_equal, rel_err  # noqa: E402

import qadam_inputs as qi  # noqa: E402

S_MODE, W_MODE = 0, 1


def _rand_grads(rng, n, d, sigma=0.01):
    return (rng.standard_normal((n, d)) * sigma).astype(np.float32)


def _run(seg, n, kg, kx, placement, T=3, grid=0, seed=0, sigma=0.01, wresid=False, x_sigma=0.2,
         split=False, options=None, **hyper):
    rng = np.random.default_rng(seed)
    d = sum(seg)
    x1 = (rng.standard_normal(d) * x_sigma).astype(np.float32)
    p = Pair(seg, n, kg, kx, placement, x1=x1, grid_g=grid, want_wresid=wresid, options=options, **hyper)
    p.compare_state()                        # first broadcast Q_x(x_1)
    for t in range(T):
        p.step(_rand_grads(rng, n, d, sigma), split_workers=split and t % 2 == 1)
        p.compare_state()
    p.close()


# ---------------------------------------------------------------- sizes: several tiles and ragged tails

@pytest.mark.parametrize("d", [1, 3, 127, 128, 129, 1023, 1024, 4096, 4097, 5000, 12289, 3 * 4096 + 640])
@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_flat_sizes(d, placement):
    _run([d], 3, 0, 0, placement, T=3, seed=d)


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_ragged_segments(placement):
    seg = [64, 129, 5000, 1, 4096, 9000, 7, 128, 4097]
    _run(seg, 4, 0, 1, placement, T=4, seed=1, wresid=True, split=True)


# ---------------------------------------------------------------- every quantizer mode

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kg,grid", [(-1, 0), (0, 0), (0, 1), (1, 0), (1, 1), (2, 0), (2, 1), (3, 0),
                                     (5, 0), (14, 0), (3, 1), (4, 1), (6, 1)])
def test_gradient_quantizer_modes(kg, grid, placement):
    _run([3000, 200, 4100], 3, kg, 0, placement, T=3, grid=grid, seed=100 + 10 * kg + grid)


@pytest.mark.parametrize("kx", [-1, 0, 1, 2, 3, 4, 5, 6, 7, 9, 10, 12, 13, 14])
def test_weight_quantizer_widths(kx):
    # x_sigma 0.4: a good share of weights falls outside [-1/2, 1/2] and is clipped
    _run([2500, 130, 4096], 2, 0, kx, S_MODE, T=2, seed=kx + 50, wresid=True, x_sigma=0.4)


@pytest.mark.parametrize("n", [1, 2, 5, 8, 16, 32, 33])
@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_worker_counts(n, placement):
    _run([6000, 300], n, 0, 0, placement, T=2, seed=n)


def test_paper_hyperparameters():
    # beta = 0.99, theta = 0.999, eps = 1e-5 (Section 5.1), moments on the workers
    _run([5000, 64, 64, 2000], 8, 0, 6, W_MODE, T=5, seed=3, beta1=0.99, beta2=0.999, eps=1e-5)
    _run([5000, 64, 64, 2000], 8, 1, 6, S_MODE, T=5, seed=4, beta1=0.99, beta2=0.999, eps=1e-5)


# ---------------------------------------------------------------- degenerate and hostile values

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_zero_gradients_and_zero_segments(placement):
    seg = [300, 4096, 50]
    p = Pair(seg, 2, 0, 0, placement, x1=np.zeros(sum(seg), np.float32))
    g = np.zeros((2, sum(seg)), np.float32)
    p.step(g)                                # every scale is 0
    p.compare_state()
    g[0, 300:300 + 4096] = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    p.step(g)                                # one live segment of one worker
    p.compare_state()
    p.close()


@pytest.mark.parametrize("kg,grid", [(0, 0), (1, 0), (2, 0), (3, 1)])
def test_ties_on_grid_values_and_tiny_magnitudes(kg, grid):
    rng = np.random.default_rng(kg)
    d = 4096 + 256
    p = Pair([d], 2, kg, 1, S_MODE, x1=np.zeros(d, np.float32), grid_g=grid)
    g = np.zeros((2, d), np.float32)
    fr = np.array([1, -1, 0.5, -0.5, 0.25, 0.75, -0.75, 0.125, 0.375, 0.625, 0.875, 0.0625, 0], np.float32)
    g[0] = rng.choice(fr, d) * np.float32(3.0)          # exact ties and on-grid values, scale 3
    g[1] = rng.choice(fr, d) * np.float32(1e-39)        # subnormal range
    g[0, 0], g[1, 0] = 3.0, 1e-39
    for _ in range(3):
        p.step(g)
        p.compare_state()
    p.close()


def test_heavy_tails_and_outliers():
    rng = np.random.default_rng(9)
    seg = [5000, 3000]
    p = Pair(seg, 3, 0, 0, S_MODE, x1=(rng.standard_normal(8000) * 0.02).astype(np.float32))
    for _ in range(4):
        g = (rng.standard_t(3, (3, 8000)) * 1e-3).astype(np.float32)
        g[rng.integers(0, 3), rng.integers(0, 8000)] = 50.0
        p.step(g)
        p.compare_state()
    p.close()


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_sparse_and_dense_code_regions(placement):
    """The server pass skips workers whose codes in a warp's rows are all level 0 and
    falls back to decoding everything where codes are dense; a vector with a dense
    third and a sparse rest, long enough that every CTA switches mode several times,
    must still match the oracle bit for bit."""
    rng = np.random.default_rng(77)
    d, n = 1 << 25, 4
    dense_end = d * 3 // 10
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    p = Pair([d], n, 0, 0, placement, x1=x1)
    for t in range(2):
        g = (rng.standard_normal((n, d)) * 1e-4).astype(np.float32)
        g[:, :dense_end] = rng.standard_normal((n, dense_end)).astype(np.float32)
        hits = rng.integers(dense_end, d, (n, 400))
        for i in range(n):
            g[i, hits[i]] = np.where(rng.random(400) < 0.5, 4.0, -4.0)
        g[:, d - 1] = 5.0
        p.step(g, threads=4)
    p.compare_state()
    p.close()


@pytest.mark.parametrize("n", [1, 4, 8, 16, 32, 33, 64])
@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_five_level_worker_counts(n, placement):
    # 3-bit codes through the pipelined server pass: unrolled (4, 8, 16, 32) and run-time worker loops
    _run([6000, 300, 3 * 2048 + 128], n, 1, 1, placement, T=2, seed=200 + n)


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_five_level_scales_whose_half_is_not_a_float(placement):
    """Five-level codes decode to scale / 2 for the inner levels.  With every scale a
    small odd multiple of the smallest subnormal that product is rounded before it is
    added (Section 5.1 defines the decoded value, the sum comes after), which a fused
    multiply-add would not reproduce; one ordinary segment rides along."""
    rng = np.random.default_rng(31)
    seg, n = [4096 + 128, 2048], 5
    d = sum(seg)
    p = Pair(seg, n, 1, 0, placement, x1=np.zeros(d, np.float32))
    tiny = np.float32(2.0 ** -149)
    for t in range(3):
        g = np.zeros((n, d), np.float32)
        k = rng.integers(-7, 8, (n, seg[0])).astype(np.float32)
        k[:, t] = np.array([7, 5, 7, 3, 5], np.float32)          # odd maxima
        g[:, :seg[0]] = k * tiny
        g[:, seg[0]:] = (rng.standard_normal((n, seg[1])) * 0.01).astype(np.float32)
        p.step(g)
        p.compare_state()
    p.close()


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_five_level_sparse_and_dense_code_regions(placement):
    rng = np.random.default_rng(78)
    d, n = 1 << 23, 8
    dense_end = d * 3 // 10
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    p = Pair([d], n, 1, 0, placement, x1=x1)
    for t in range(2):
        g = (rng.standard_normal((n, d)) * 1e-4).astype(np.float32)
        g[:, :dense_end] = rng.standard_normal((n, dense_end)).astype(np.float32)
        hits = rng.integers(dense_end, d, (n, 300))
        for i in range(n):
            g[i, hits[i]] = rng.choice(np.array([4.0, -4.0, 2.0, -2.0], np.float32), 300)
        g[:, d - 1] = 5.0
        p.step(g, threads=4)
    p.compare_state()
    p.close()


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kg,grid", [(2, 0), (2, 1), (3, 1), (6, 1), (14, 0)])
@pytest.mark.parametrize("n", [1, 16, 33])
def test_table_decoded_grids(kg, grid, n, placement):
    """Grids beyond five levels go through the server pipeline's table decode: 3, 4, 5, 8 and
    5 bits per code here, fields that straddle 32-bit words, several tiles and a ragged tail."""
    _run([3 * 2048 + 640, 130, 4096], n, kg, 1, placement, T=2, grid=grid, seed=500 + 7 * kg + grid + n)


def test_table_decoded_grid_sparse_and_dense_regions():
    rng = np.random.default_rng(79)
    d, n = 1 << 22, 8
    dense_end = d * 3 // 10
    p = Pair([d], n, 3, 0, S_MODE, x1=(rng.standard_normal(d) * 0.05).astype(np.float32))
    for t in range(2):
        g = (rng.standard_normal((n, d)) * 1e-5).astype(np.float32)
        g[:, :dense_end] = rng.standard_normal((n, dense_end)).astype(np.float32)
        hits = rng.integers(dense_end, d, (n, 300))
        for i in range(n):
            g[i, hits[i]] = rng.choice(np.array([4.0, -4.0, 1.0, -0.5], np.float32), 300)
        g[:, d - 1] = 5.0
        p.step(g, threads=4)
    p.compare_state()
    p.close()


# ---------------------------------------------------------------- the on-chip worker kernel

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_on_chip_worker_many_small_tensors(placement):
    # hundreds of (worker, segment) pairs of one or two tiles: streaks of a single tile,
    # CTAs that own nothing of a pair, pairs that end in the middle of a tile row
    rng = np.random.default_rng(11)
    seg = [int(v) for v in rng.integers(1, 6000, size=400)]
    _run(seg, 3, 0, 0, placement, T=3, seed=12)
    _run(seg[:150], 5, 1, 1, placement, T=2, seed=13)


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_on_chip_worker_rings_wrap(placement):
    # more than 32 tiles per CTA: the rings of slots, stages and tile headers all go round
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    per_seg = sms * 5 * 4096 + 4096 + 300            # 6 tiles for some CTAs, a ragged tail
    _run([per_seg, 5000, per_seg, 77, per_seg], 3, 0, 0, placement, T=3, seed=14)


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_on_chip_worker_capacity_boundary(placement):
    # tensors around the largest pair the on-chip kernel takes: the kernel and the two
    # streaming launches share one step, each over its own tile table
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rng = np.random.default_rng(15)
    tile = 4096
    # around slots - spare for a 227 KB SM: 12 - 2 (moments on the server), 8 - 2 (on the workers)
    lo = 10 if placement == S_MODE else 6
    for slots_used in (lo, lo + 1, lo + 2):
        cap = sms * slots_used * tile
        seg = [cap, 300, cap + tile, 70000, cap - tile + 1]
        n, d = 2, sum([cap, 300, cap + tile, 70000, cap - tile + 1])
        x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
        p = Pair(seg, n, 0, 0, placement, x1=x1)
        one, two = p.gpu.worker_pass_model()
        assert one + two == n * p.gpu.D
        for t in range(2):
            p.step(_rand_grads(rng, n, d))
            p.compare_state()
        p.close()
        if slots_used == lo:
            assert one > 0, "no pair took the on-chip kernel"
        if slots_used == lo + 2:
            assert two > 0, "no pair took the streaming launches"


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kx", [0, 3, 6, 9, -1])
def test_on_chip_worker_l2_term_many_tiles(kx, placement):
    # the l2 term inside the on-chip kernel with several tiles per CTA: the held-weight
    # codes of a tile are fetched while the tile before it is processed (widths up to 8
    # bits); wider codes and unquantized weights are read in place
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    seg = [sms * 3 * 4096 + 300, 5000, 70000, 129]
    n, d = 3, sum([sms * 3 * 4096 + 300, 5000, 70000, 129])
    rng = np.random.default_rng(40 + kx)
    x1 = (rng.standard_normal(d) * 0.3).astype(np.float32)
    p = Pair(seg, n, 0, kx, placement, x1=x1)
    for lam in (5e-4, 0.05, 0.0):
        p.set_regularization(lam)
        p.step(_rand_grads(rng, n, d))
        p.compare_state()
    p.close()


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_on_chip_worker_counter_hand_over(placement):
    # the on-chip kernel hands a pair's scale over through one word per (pair, CTA) while the
    # workspace has room for them, else through one counter per pair; the hand_over option
    # forces the second route
    import paper_2004_14180_b200 as qb
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    seg = [sms * 2 * 4096 + 300, 5000, 64, 70000, 129]
    _run(seg, 3, 0, 0, placement, T=3, seed=90 + placement,
         options=qb.QAdamOptions(hand_over=qb.HANDOVER_COUNTERS))


@pytest.mark.parametrize("hand_over", ["auto", "counters"])
@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_on_chip_worker_one_tile_pairs(placement, hand_over):
    # pairs of a single tile take their scale from the tile's header inside the CTA; here
    # each CTA gets more than 32 of them in a row (the ring of headers goes round), with
    # pairs of several tiles in between, with and without the l2 term
    import paper_2004_14180_b200 as qb
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    sizes = (4096, 2048, 100, 4095, 1)
    seg = [sizes[k % len(sizes)] for k in range(sms * 34)]
    seg[sms * 7] = 3 * 4096 + 5
    seg[sms * 20 + 3] = sms * 4096 + 77
    n, d = 2, sum(seg)
    rng = np.random.default_rng(120 + placement)
    x1 = (rng.standard_normal(d) * 0.3).astype(np.float32)
    opt = qb.QAdamOptions(hand_over=qb.HANDOVER_COUNTERS) if hand_over == "counters" else None
    p = Pair(seg, n, 0, 0, placement, x1=x1, options=opt)
    one, two = p.gpu.worker_pass_model()
    assert two == 0, "every pair fits on chip"
    for lam in (0.0, 5e-4):
        p.set_regularization(lam)
        p.step(_rand_grads(rng, n, d))
        p.compare_state()
    p.close()


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_streaming_launches_only(placement):
    # worker_kernel = STREAMING sends every pair through the two streaming launches, the
    # route that otherwise only pairs too large for the chip, partial worker ranges and some
    # l2 cases take
    import paper_2004_14180_b200 as qb
    rng = np.random.default_rng(70 + placement)
    seg = [9000, 64, 129, 3 * 4096 + 640, 1, 70000]
    n, d = 4, sum([9000, 64, 129, 3 * 4096 + 640, 1, 70000])
    x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
    p = Pair(seg, n, 0, 1, placement, x1=x1, options=qb.QAdamOptions(worker_kernel=qb.WORKER_STREAMING))
    one, two = p.gpu.worker_pass_model()
    assert one == 0 and two == n * p.gpu.D
    for t in range(3):
        p.step(_rand_grads(rng, n, d))
        p.compare_state()
    p.close()


# ---------------------------------------------------------------- l2 term and step-dependent rates

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kg,kx", [(0, 0), (1, 1), (0, 6), (2, 2), (0, -1), (-1, 0), (0, 4), (0, 10), (0, 14)])
def test_l2_term(kg, kx, placement):
    """Section 5.1's weight decay: g + lambda * (weights the workers hold), for every width of
    the packed broadcast the workers decode (2, 3, 4, 6, 8, 12, 16 bits) and for unquantized
    weights, switched on after one plain step and off again at the end."""
    rng = np.random.default_rng(300 + 10 * kg + kx)
    seg, n = [3000, 200, 4100, 64], 3
    d = sum(seg)
    x1 = (rng.standard_normal(d) * 0.3).astype(np.float32)
    p = Pair(seg, n, kg, kx, placement, x1=x1)
    lam = [0.0, 5e-4, 5e-4, 0.1, 0.0]
    for t in range(5):
        p.set_regularization(lam[t])
        p.step(_rand_grads(rng, n, d), split_workers=t == 2)
        p.compare_state()
    p.close()


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
def test_step_dependent_rates(placement):
    """Assumption 2: theta_t = 1 - theta/t, alpha_t = alpha/sqrt(t), a decaying beta_t."""
    rng = np.random.default_rng(41)
    seg, n = [5000, 130], 4
    d = sum(seg)
    p = Pair(seg, n, 0, 0, placement, x1=(rng.standard_normal(d) * 0.1).astype(np.float32))
    for t in range(1, 7):
        p.set_moment_rates(float(np.float32(0.9 * 0.8 ** (t - 1))), float(np.float32(1.0 - 0.5 / t)))
        p.step(_rand_grads(rng, n, d), lr=float(np.float32(1e-3 / np.sqrt(t))))
        p.compare_state()
    p.close()


def test_setters_reject_bad_values():
    import paper_2004_14180_b200 as qb
    q = qb.QAdam([1000], 1, kg=0, kx=0)
    for bad in [(1.0, 0.5), (-0.1, 0.5), (0.5, 1.0), (0.5, float("nan"))]:
        with pytest.raises(qb.QAdamError):
            q.set_moment_rates(*bad)
    for bad in [-1e-3, float("inf"), float("nan")]:
        with pytest.raises(qb.QAdamError):
            q.set_regularization(bad)
    q.close()


def test_nonfinite_input_sets_status_bit():
    import paper_2004_14180_b200 as qb
    q = qb.QAdam([1000], 1, kg=0, kx=-1)
    g = torch.zeros(1, q.D, device="cuda")
    g[0, 5] = float("inf")
    q.worker_compress(1, g)
    assert q.poll_status() & qb.ST_NONFINITE
    q.close()


# ---------------------------------------------------------------- the configurations, at their sizes

def _run_workload(w, steps, placement, threads=8, exact=True):
    x1 = qi.initial_weights(w, "cpu").numpy()
    p = Pair(w.scale_seg_len, w.n, w.kg, w.kx, placement, x1=x1,
             beta1=w.beta1, beta2=w.beta2, eps=w.eps, lr=w.lr)
    for t in range(1, steps + 1):
        g = np.stack([qi.gradients(w, t, i, "cpu").numpy() for i in range(w.n)])
        p.step(g, threads=threads)
    p.compare_state(exact=exact)
    ratio = p.gpu.compression_ratio()
    p.close()
    return ratio


def test_config_flat20_all_steps():
    w = qi.get_workload("flat20")
    ratio = _run_workload(w, w.steps, S_MODE)
    assert abs(ratio - 16.0) < 0.01                       # 32-bit -> 2-bit codes
    _run_workload(w, w.steps, W_MODE)


@pytest.mark.parametrize("name", ["resnet18_qg", "resnet18_qg_qx_k0", "resnet18_qg_qx_k1",
                                  "resnet18_qg_qx_8bit"])
def test_config_resnet18_shaped(name):
    w = qi.get_workload(name)
    ratio = _run_workload(w, 4, S_MODE)
    want = 32.0 / (2 if w.kg == 0 else 3)
    assert abs(ratio / want - 1) < 0.01                   # per-tensor scales and padding cost < 1 %


def test_config_resnet18_shaped_paper_placement_and_single_scale():
    w = qi.get_workload("resnet18_qg_qx_k0")
    _run_workload(w, 3, W_MODE)
    _run_workload(w.with_(per_tensor_scale=False), 3, S_MODE)


def test_config_resnet18_shaped_all_steps():
    """The ResNet-18-shaped workload over its full T = 100 steps (gradient and weight
    quantizers on, moments on the server): codes and scales compared after every step, the
    whole state every tenth step and at the end.  Gradients are drawn on the GPU."""
    w = qi.get_workload("resnet18_qg_qx_k0")
    dev = torch.device("cuda")
    x1 = qi.initial_weights(w, "cpu").numpy()
    p = Pair(w.scale_seg_len, w.n, w.kg, w.kx, S_MODE, x1=x1, beta1=w.beta1, beta2=w.beta2, eps=w.eps, lr=w.lr)
    for t in range(1, w.steps + 1):
        g = torch.stack([qi.gradients(w, t, i, dev) for i in range(w.n)]).cpu().numpy()
        p.step(g, threads=8)
        if t % 10 == 0:
            p.compare_state()
    assert p.step_no == 100
    p.close()


# ---------------------------------------------------------------- the plain server kernel

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kg,grid", [(0, 0), (1, 0), (3, 0), (3, 1)])
@pytest.mark.parametrize("n", [65, 128])
def test_plain_server_kernel_many_workers(n, kg, grid, placement):
    """More than 64 workers go through the grid-stride server kernel (its own ternary decode
    and its per-worker table of level values for the other grids): several tiles, a ragged
    tail, two segments with different scales."""
    _run([3 * 4096 + 640, 130, 4096], n, kg, 1, placement, T=2, grid=grid, seed=700 + n + 10 * kg + grid)


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kg", [0, 1, 3])
def test_plain_server_kernel_sparse_and_dense_regions(kg, placement):
    # the same kernel chosen by option at a worker count the pipelined pass would take,
    # over a vector with a dense third and a sparse rest
    import paper_2004_14180_b200 as qb
    rng = np.random.default_rng(80 + kg)
    d, n = 1 << 21, 6
    dense_end = d * 3 // 10
    x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    p = Pair([d], n, kg, 0, placement, x1=x1, options=qb.QAdamOptions(server_kernel=qb.SERVER_PLAIN))
    for t in range(2):
        g = (rng.standard_normal((n, d)) * 1e-4).astype(np.float32)
        g[:, :dense_end] = rng.standard_normal((n, dense_end)).astype(np.float32)
        hits = rng.integers(dense_end, d, (n, 300))
        for i in range(n):
            g[i, hits[i]] = rng.choice(np.array([4.0, -4.0, 2.0, -1.0], np.float32), 300)
        g[:, d - 1] = 5.0
        p.step(g, threads=4)
        p.compare_state()
    p.close()


@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("density", [1e-4, 1e-3, 1e-2, 0.1])
def test_pipelined_server_code_densities(density, placement):
    """The pipelined pass decodes only the workers that have a non-zero code in a warp's 256
    elements and switches to the unrolled loop over all workers when most do: densities on
    both sides of that switch, n = 16 (compile-time worker count) and n = 5 (run-time)."""
    rng = np.random.default_rng(int(density * 1e6) + placement)
    d = 3 * (1 << 18) + 640
    for n in (16, 5):
        x1 = (rng.standard_normal(d) * 0.05).astype(np.float32)
        p = Pair([d], n, 0, 0, placement, x1=x1)
        for t in range(2):
            g = (rng.standard_normal((n, d)) * 1e-6).astype(np.float32)
            hit = rng.random((n, d)) < density
            g[hit] = np.where(rng.random(int(hit.sum())) < 0.5, 1.0, -1.0).astype(np.float32)
            g[:, 0] = 1.5
            p.step(g, threads=4)
            p.compare_state()
        p.close()


# ---------------------------------------------------------------- the stochastic ternary operator

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("n,seed", [(3, 1), (16, (1 << 63) + 12345), (70, 20200429)])
def test_stochastic_ternary_operator(n, seed, placement):
    """The comparison operator of Section 5.1 (level 1 with probability |u| / max|u|): both
    sides draw their coins from Philox4x32-10 with counter (element / 4, worker, step) and key
    = seed, so codes are bit-identical; several tiles, ragged tails, partial worker calls,
    the pipelined and the plain server pass, with the l2 term switched on for one step."""
    rng = np.random.default_rng(900 + n)
    seg = [3 * 4096 + 640, 130, 70000, 1]
    d = sum(seg)
    x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
    p = Pair(seg, n, 0, 1, placement, x1=x1, grid_g=2, seed=seed)
    assert p.gpu.worker_pass_model()[0] == 0          # this operator runs in the streaming launches
    lam = [0.0, 0.0, 5e-4, 0.0]
    for t in range(4):
        p.set_regularization(lam[t])
        p.step(_rand_grads(rng, n, d), split_workers=t == 1)
        p.compare_state()
    live = np.mean(p.cpu.gcodes != 0x55)
    assert live > 0.2                                  # far denser than the deterministic ternary codes
    p.close()


def test_stochastic_operator_is_ternary_only():
    import paper_2004_14180_b200 as qb
    with pytest.raises(qb.QAdamError) as ei:
        qb.QAdam([1000], 2, kg=1, grid_g=qb.GRID_STOCHASTIC)
    assert ei.value.code == -3
    with pytest.raises(qb.QAdamError):
        qb.QAdam([1000], 2, kg=-1, grid_g=qb.GRID_STOCHASTIC)


# ---------------------------------------------------------------- the step from host buffers

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kx", [0, -1])
def test_step_from_host_buffers(kx, placement):
    """qadam_step_host (pinned host gradients in, worker by worker on a copy stream; packed
    broadcast or x out) gives the bits of the two-call step and of the oracle."""
    rng = np.random.default_rng(60 + kx + placement)
    seg, n = [3 * 4096 + 640, 130, 70000, 1], 5
    d = sum(seg)
    x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
    p = Pair(seg, n, 0, kx, placement, x1=x1)
    D = p.gpu.D
    g_stage = torch.zeros(n, D, device="cuda")
    out_bytes = p.gpu.wcode_bytes if kx >= 0 else 4 * D
    out_host = torch.zeros(out_bytes, dtype=torch.uint8).pin_memory()
    for t in range(1, 4):
        gp = p.cpu.to_padded(_rand_grads(rng, n, d))
        g_host = torch.from_numpy(gp).pin_memory()
        p.gpu.step_host(t, g_host.view(-1), g_stage, out_host)
        p.cpu.step(gp, p.lr)
        p.step_no = t
        p.compare_worker_outputs()
        p.compare_state()
        want = p.cpu.wcodes if kx >= 0 else p.cpu.x.view(np.uint8)
        assert np.array_equal(out_host.numpy()[:want.size], want)
    p.close()


# ---------------------------------------------------------------- error buffer for the broadcast

@pytest.mark.parametrize("placement", [S_MODE, W_MODE])
@pytest.mark.parametrize("kx,n,kg", [(0, 4, 0), (3, 5, 0), (6, 16, 1), (0, 70, 0), (2, 3, 3)])
def test_weight_feedback_buffer(kx, n, kg, placement):
    """The optional error buffer of the broadcast (Q_x applied to x + e^w, e^w <- what Q_x
    dropped; not in the paper): through the pipelined pass with its ternary-weight path, the
    generic path, the table decode and the plain kernel, one step served by ranges."""
    import paper_2004_14180_b200 as qb
    rng = np.random.default_rng(1200 + 10 * kx + n)
    seg = [3 * 4096 + 640, 130, 9000, 1]
    d = sum(seg)
    x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
    p = Pair(seg, n, kg, kx, placement, x1=x1, want_wfeedback=True, want_wresid=(kx == 3))
    p.compare_state()                                   # the first broadcast already feeds the buffer
    for t in range(1, 5):
        g = _rand_grads(rng, n, d)
        if t == 3:                                      # one step range by range
            gp = p.cpu.to_padded(g)
            p.gpu.worker_compress(t, torch.from_numpy(gp).cuda())
            p.cpu.workers_step(gp, p.lr)
            cuts = p.gpu.shard_cuts(3)
            for r in (2, 0, 1):
                p.gpu.server_step_range(t, cuts[r], cuts[r + 1])
            p.gpu.finish_step(t)
            p.cpu.server_step(p.lr)
            p.step_no = t
        else:
            p.step(g)
        p.compare_state()
    assert float(p.gpu.wfeedback.abs().max()) > 0
    p.close()
    with pytest.raises(qb.QAdamError) as ei:
        qb.QAdam([1000], 2, kg=0, kx=-1, want_wfeedback=True)      # nothing to feed back without Q_x
    assert ei.value.code == -3


def test_ternary_decision_around_the_sliver_and_at_the_ends_of_the_fast_range():
    """The ternary level is decided without a division outside the sliver (s/2, (s/2)(1 + 2^-21)]
    and by saturating fp32 differences: every float within 12 ulps of both ends of the sliver,
    both signs, for an ordinary scale, for scales at the two ends of the range that takes the
    fast path (1.1e-30, 2.9e38) and just outside it (0.9e-30: the division decides everything).
    Worker side only, moments on the server, e = 0, so that u is exactly the value planted (the
    server's average of such scales would overflow)."""
    d, n = 4096 + 512, 4
    scales = np.array([1.0, 1.1e-30, 2.9e38, 0.9e-30], np.float32)
    g = np.zeros((n, d), np.float32)
    rng = np.random.default_rng(5)
    for i, s in enumerate(scales):
        half = np.float32(0.5) * s
        hi = half * np.float32(1.0 + 2.0 ** -21)
        vals = []
        for base in (half, hi):
            v = base
            for _ in range(12):
                v = np.nextafter(v, np.float32(0))
            for _ in range(25):
                vals.append(v)
                v = np.nextafter(v, np.float32(np.inf))
        vals = np.array(vals, np.float32)
        row = rng.choice(np.concatenate([vals, -vals, np.float32([0.0]), half * np.float32([0.25, 0.9, 1.5, 1.99])]), d)
        row[0] = s                                           # the scale itself
        g[i] = row.astype(np.float32)
    for options in (None, "streaming"):
        import paper_2004_14180_b200 as qb
        opt = qb.QAdamOptions(worker_kernel=qb.WORKER_STREAMING) if options else None
        p = Pair([d], n, 0, 0, S_MODE, x1=np.zeros(d, np.float32), options=opt)
        gp = p.cpu.to_padded(g)
        p.gpu.worker_compress(1, torch.from_numpy(gp).cuda())
        p.cpu.workers_step(gp, p.lr)
        p.compare_worker_outputs()
        assert np.array_equal(p.cpu.scales[:, 0], scales)
        assert bits_equal(p.gpu.e.cpu().numpy(), p.cpu.e), "e differs"
        # some values of every worker fall on either side, and inside the sliver
        codes = p.cpu.gcodes
        assert (codes != 0x55).any(axis=1).all()
        p.close()


def test_five_level_decision_around_both_midpoints_and_at_the_ends_of_the_fast_range():
    """The five-level index [y > 1/4] + [y > 3/4] is settled from |u| * fl(1/s) by saturating
    fp32 differences unless that product lies within 2^-20 (relative) of a midpoint, where the
    division decides: every float within 12 ulps of s/4 and 3s/4 and of the two ends of either
    band, both signs, for an ordinary scale, an awkward one (1/3: its reciprocal is rounded), and
    scales at the two ends of the range that takes the fast path and just outside it.  Worker
    side only, moments on the server, e = 0, so that u is exactly the value planted."""
    import paper_2004_14180_b200 as qb
    d, n = 4096 + 512, 5
    scales = np.array([1.0, 1.0 / 3.0, 1.1e-30, 2.9e38, 0.9e-30], np.float32)
    g = np.zeros((n, d), np.float32)
    rng = np.random.default_rng(6)
    for i, s in enumerate(scales):
        vals = []
        for t in (0.25, 0.75):
            mid = np.float32(t) * s
            for base in (mid * np.float32(1.0 - 2.0 ** -20), mid, mid * np.float32(1.0 + 2.0 ** -20)):
                v = np.float32(base)
                for _ in range(12):
                    v = np.nextafter(v, np.float32(0))
                for _ in range(25):
                    vals.append(v)
                    v = np.nextafter(v, np.float32(np.inf))
        vals = np.array(vals, np.float32)
        extra = s * np.float32([0.0, 0.1, 0.24, 0.26, 0.5, 0.74, 0.76, 0.99])
        row = rng.choice(np.concatenate([vals, -vals, extra, -extra]), d)
        row[0] = s                                           # the scale itself
        g[i] = row.astype(np.float32)
    for options in (None, "streaming"):
        opt = qb.QAdamOptions(worker_kernel=qb.WORKER_STREAMING) if options else None
        p = Pair([d], n, 1, 0, S_MODE, x1=np.zeros(d, np.float32), options=opt)
        gp = p.cpu.to_padded(g)
        p.gpu.worker_compress(1, torch.from_numpy(gp).cuda())
        p.cpu.workers_step(gp, p.lr)
        p.compare_worker_outputs()
        assert np.array_equal(p.cpu.scales[:, 0], scales)
        assert bits_equal(p.gpu.e.cpu().numpy(), p.cpu.e), "e differs"
        p.close()
