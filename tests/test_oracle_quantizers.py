"""Pins of the oracle's quantizers and packers against things other than itself:
hand-worked fixtures, exact brute force over the level set, invariants the
paper states (Assumptions 2 and 3), and the byte ratios of its tables."""
import numpy as np
import pytest

from _util import (brute_qg, brute_qx, level_fractions, pack_little_endian, read_golden)


# ---------------------------------------------------------------- hand-worked

def test_ternary_hand_example(oracle):
    gold = read_golden("ternary_example.txt")
    u = np.array(gold["u"], np.float32)
    s, q, r = oracle.quantize_grad_segment(u, kg=0)
    assert s == gold["scale"][0]
    assert q.tolist() == [int(v) for v in gold["q"]]
    assert np.array_equal(r, np.array(gold["resid"], np.float32))
    deq = u - r            # exact here: every value is a small dyadic number
    assert deq.tolist() == gold["deq"]
    packed = oracle.pack_bits((q + 1).astype(np.uint32), bits=2)
    assert packed.tolist() == [int(v) for v in gold["packed"]]
    # both grid readings coincide for k = 0
    s1, q1, r1 = oracle.quantize_grad_segment(u, kg=0, grid=oracle.GRID_UNIFORM)
    assert (s1, q1.tolist(), r1.tolist()) == (s, q.tolist(), r.tolist())


def test_five_level_hand_example(oracle):
    gold = read_golden("five_level_example.txt")
    u = np.array(gold["u"], np.float32)
    for grid in (oracle.GRID_POW2, oracle.GRID_UNIFORM):
        s, q, r = oracle.quantize_grad_segment(u, kg=1, grid=grid)
        assert s == gold["scale"][0]
        assert q.tolist() == [int(v) for v in gold["q"]]
        assert np.array_equal(r, np.array(gold["resid"], np.float32))
        assert (u - r).tolist() == gold["deq"]


def test_weight_grid_hand_example(oracle):
    gold = read_golden("weight_grid_example.txt")
    x = np.array(gold["x"], np.float32)
    q, xh, r = oracle.quantize_weights(x, kx=1)
    assert q.tolist() == [int(v) for v in gold["q"]]
    assert xh.tolist() == gold["xhat"]
    assert np.array_equal(r, x - xh)


# ---------------------------------------------------------------- level sets

@pytest.mark.parametrize("k", [0, 1, 2, 3, 5])
@pytest.mark.parametrize("grid", [0, 1])
def test_level_sets_match_definition(oracle, k, grid):
    lv = oracle.grad_levels(k, grid)
    want = [float(f) for f in level_fractions(k, grid)]
    assert lv.tolist() == want
    n_codes = 2 * (len(lv) - 1) + 1
    assert oracle.grad_code_bits(k, grid) == int(np.ceil(np.log2(n_codes)))


def test_code_widths_of_the_tables(oracle):
    # 3 levels -> 2 bits, 5 levels -> 3 bits (Comm column: 32 -> 3 -> 2 bits)
    assert oracle.grad_code_bits(0) == 2
    assert oracle.grad_code_bits(1) == 3
    # 2^(k+1)+1 weight levels -> k+2 bits; 8 and 16 bits are the Size column's
    assert oracle.weight_code_bits(0) == 2
    assert oracle.weight_code_bits(1) == 3
    assert oracle.weight_code_bits(6) == 8
    assert oracle.weight_code_bits(14) == 16
    gold = read_golden("table_bytes.txt")
    for t in ("table1", "table2"):
        full, three_bit, two_bit = gold[t + "_comm"]
        assert abs(full / two_bit - 32 / oracle.grad_code_bits(0)) < 0.02
        assert abs(full / three_bit - 32 / oracle.grad_code_bits(1)) < 0.02
        full, sixteen, eight = gold[t + "_size"]
        assert abs(full / eight - 32 / oracle.weight_code_bits(6)) < 0.02
        assert abs(full / sixteen - 32 / oracle.weight_code_bits(14)) < 0.02


# ---------------------------------------------------------------- brute force

def _tricky_vectors(rng, d):
    """Vectors with exact ties, on-grid values, zeros, repeated maxima, subnormals."""
    out = []
    base = rng.standard_normal(d).astype(np.float32)
    out.append(base)
    v = base.copy()
    s = np.max(np.abs(v))
    for j, frac in enumerate((0.5, -0.5, 0.25, -0.75, 0.125, 0.375, 1.0, -1.0, 0.0)):
        if j < d:
            v[j] = np.float32(frac) * s
    out.append(v)
    out.append(np.zeros(d, np.float32))
    out.append(np.full(d, -3.5, np.float32))
    out.append((rng.standard_normal(d) * 1e-42).astype(np.float32))      # subnormal range
    out.append((rng.standard_t(3, d) * 1e-3).astype(np.float32))          # heavy tails
    one = np.zeros(d, np.float32)
    one[d // 2] = -7.25
    out.append(one)
    return out


@pytest.mark.parametrize("k,grid", [(0, 0), (1, 0), (1, 1), (2, 0), (2, 1), (3, 0), (3, 1), (5, 1)])
def test_qg_equals_exact_nearest_level(oracle, k, grid):
    rng = np.random.default_rng(100 + 7 * k + grid)
    for d in (1, 2, 5, 16):
        for u in _tricky_vectors(rng, d):
            s, q, r = oracle.quantize_grad_segment(u, k, grid)
            bs, bq = brute_qg(u, k, grid)
            assert s == bs
            assert q.tolist() == bq.tolist(), (u, k, grid)


def test_qg_random_brute_force_larger(oracle):
    rng = np.random.default_rng(5)
    for k, grid in ((0, 0), (1, 0), (2, 0), (2, 1)):
        u = (rng.standard_normal(3000) * 10.0 ** rng.uniform(-6, 2)).astype(np.float32)
        s, q, r = oracle.quantize_grad_segment(u, k, grid)
        bs, bq = brute_qg(u, k, grid)
        assert s == bs and np.array_equal(q, bq)


@pytest.mark.parametrize("kx", [0, 1, 2, 6])
def test_qx_equals_exact_nearest_grid_point(oracle, kx):
    rng = np.random.default_rng(kx)
    x = np.concatenate([
        rng.standard_normal(400).astype(np.float32) * 0.3,
        rng.uniform(-0.5, 0.5, 400).astype(np.float32),
        # every grid point, every midpoint (tie), and their float neighbours
        np.array([c / 2 ** (kx + 2) for c in range(-2 ** (kx + 1) - 4, 2 ** (kx + 1) + 5)], np.float32),
    ])
    ties = np.array([c / 2 ** (kx + 2) for c in range(-2 ** (kx + 1), 2 ** (kx + 1) + 1)], np.float32)
    x = np.concatenate([x, np.nextafter(ties, np.float32(1)), np.nextafter(ties, np.float32(-1)),
                        np.array([0.0, -0.0, 1e-30, -1e-42, 5.0, -80.0, 3e38], np.float32)])
    q, xh, r = oracle.quantize_weights(x, kx)
    assert np.array_equal(q, brute_qx(x, kx))
    assert np.array_equal(xh, q.astype(np.float64) / 2 ** (kx + 1))
    assert np.array_equal(r, x - xh)


# ---------------------------------------------------------------- invariants

@pytest.mark.parametrize("k,grid", [(0, 0), (1, 0), (3, 0), (3, 1), (6, 1)])
def test_qg_invariants(oracle, k, grid):
    rng = np.random.default_rng(11 + k)
    lv = oracle.grad_levels(k, grid)
    L = len(lv) - 1
    gaps = np.diff(lv.astype(np.float64))
    for d in (1, 3, 128, 1000, 4097):
        u = (rng.standard_normal(d) * 0.02).astype(np.float32)
        s, q, r = oracle.quantize_grad_segment(u, k, grid)
        # codes within the stated levels
        assert q.min() >= -L and q.max() <= L
        # the max-abs element sits on the top level and is reconstructed exactly
        jmax = int(np.argmax(np.abs(u)))
        assert abs(q[jmax]) == L and r[jmax] == 0.0
        # error is at most half the widest gap times the scale, and never exceeds |u|
        assert np.all(np.abs(r.astype(np.float64)) <= s * gaps.max() / 2 * (1 + 1e-6))
        assert np.all(np.abs(r) <= np.abs(u))
        # contraction (Assumption 2): |u - Q(u)| < |u| for u != 0
        assert np.linalg.norm(r.astype(np.float64)) < np.linalg.norm(u.astype(np.float64))
        # sign of a non-zero code matches the sign of the input
        nz = q != 0
        assert np.all(np.sign(q[nz]) == np.sign(u[nz]))


@pytest.mark.parametrize("k,grid", [(0, 0), (1, 0), (2, 0), (2, 1), (4, 1)])
def test_qg_reconstructs_on_grid_inputs_exactly(oracle, k, grid):
    rng = np.random.default_rng(3)
    lv = oracle.grad_levels(k, grid)
    L = len(lv) - 1
    for s in (np.float32(1.0), np.float32(0.0371), np.float32(123.456)):
        c = rng.integers(-L, L + 1, 257)
        c[0] = L                                     # make sure the top level is present
        u = np.sign(c).astype(np.float32) * (s * lv[np.abs(c)])   # fl(s * level), signed
        s_out, q, r = oracle.quantize_grad_segment(u, k, grid)
        assert s_out == s
        assert np.array_equal(q, c)
        assert not r.any()


def test_qg_zero_vector(oracle):
    s, q, r = oracle.quantize_grad_segment(np.zeros(9, np.float32), 0)
    assert s == 0.0 and not q.any() and not r.any()


@pytest.mark.parametrize("kx", [0, 1, 3, 6, 14])
def test_qx_error_bound_and_range(oracle, kx):
    # Assumption 3 with delta_x = 2^-(kx+2) per coordinate, for |x| <= 1/2
    rng = np.random.default_rng(kx)
    x = rng.uniform(-0.5, 0.5, 5000).astype(np.float32)
    q, xh, r = oracle.quantize_weights(x, kx)
    assert np.all(np.abs(r.astype(np.float64)) <= 2.0 ** -(kx + 2))
    assert q.min() >= -2 ** kx and q.max() <= 2 ** kx
    # the residual is exact, so the master copy is recovered from broadcast + residual
    assert np.array_equal(xh + r, x)
    # clipping outside the grid
    q2, xh2, _ = oracle.quantize_weights(np.array([0.9, -7.0], np.float32), kx)
    assert xh2.tolist() == [0.5, -0.5]


# ---------------------------------------------------------------- packing

@pytest.mark.parametrize("bits", [2, 3, 4, 5, 7, 8, 11, 16])
def test_pack_is_little_endian_bit_string_and_round_trips(oracle, bits):
    rng = np.random.default_rng(bits)
    for count in (1, 7, 128, 1000):
        codes = rng.integers(0, 2 ** bits, count).astype(np.uint32)
        packed = oracle.pack_bits(codes, bits)
        assert packed.size == (count * bits + 7) // 8
        assert np.array_equal(packed, pack_little_endian(codes, bits))
        assert np.array_equal(oracle.unpack_bits(packed, count, bits), codes)


def test_two_bit_packing_against_numpy_bit_order(oracle):
    rng = np.random.default_rng(0)
    codes = rng.integers(0, 3, 4096).astype(np.uint32)
    bits = np.stack([(codes >> 0) & 1, (codes >> 1) & 1], axis=1).astype(np.uint8).reshape(-1)
    assert np.array_equal(oracle.pack_bits(codes, 2), np.packbits(bits, bitorder="little"))
