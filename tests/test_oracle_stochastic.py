"""Pins of the oracle's random stream and of the stochastic ternary operator built on it.

Philox4x32-10 is checked against a restatement of its published definition in Python's
unbounded integers (written apart from the oracle's C++), against the Philox routine of the
Triton package run by its CPU interpreter (a library routine, when it can be loaded), and
through properties a wrong round function would break (it is a bijection of the counter;
one flipped input bit flips half of the output bits).  The operator is checked against its
definition coordinate by coordinate, for unbiasedness over a million coins, and for what it
must never do (drop the arg-max, raise a zero)."""
import os

import numpy as np
import pytest

M32 = (1 << 32) - 1


def philox_bigint(ctr, key, rounds=10):
    """Ten rounds of Philox-4x32 over Python integers: every step is the arithmetic of the
    definition (full 64-bit products, explicit masks), nothing borrowed from the oracle."""
    c = [int(v) & M32 for v in ctr]
    k = [int(v) & M32 for v in key]
    for _ in range(rounds):
        prod_a = 0xD2511F53 * c[0]
        prod_b = 0xCD9E8D57 * c[2]
        c = [((prod_b >> 32) ^ c[1] ^ k[0]) & M32, prod_b & M32,
             ((prod_a >> 32) ^ c[3] ^ k[1]) & M32, prod_a & M32]
        k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
    return c


def test_philox_matches_the_definition_in_big_integers(oracle):
    rng = np.random.default_rng(1)
    cases = [([0, 0, 0, 0], [0, 0]), ([M32] * 4, [M32] * 2), ([1, 0, 0, 0], [0, 0]), ([0, 0, 0, 0], [1, 0])]
    cases += [(rng.integers(0, 1 << 32, 4).tolist(), rng.integers(0, 1 << 32, 2).tolist()) for _ in range(300)]
    for ctr, key in cases:
        assert oracle.philox4x32_10(ctr, key).tolist() == philox_bigint(ctr, key), (ctr, key)


def test_philox_matches_the_triton_library_routine(oracle):
    os.environ.setdefault("TRITON_INTERPRET", "1")
    if os.environ["TRITON_INTERPRET"] != "1":
        pytest.skip("the Triton interpreter is switched off")
    triton = pytest.importorskip("triton")
    import torch
    import triton.language as tl
    if not hasattr(tl, "philox_impl"):
        pytest.skip("this Triton has no philox_impl")

    @triton.jit
    def block_kernel(out_ptr, c_ptr, k0, k1, N: tl.constexpr):
        offs = tl.arange(0, N)
        c0 = tl.load(c_ptr + offs)
        c1 = tl.load(c_ptr + N + offs)
        c2 = tl.load(c_ptr + 2 * N + offs)
        c3 = tl.load(c_ptr + 3 * N + offs)
        key0 = tl.full((N,), 0, tl.uint32) + k0
        key1 = tl.full((N,), 0, tl.uint32) + k1
        a, b, c, d = tl.philox_impl(c0, c1, c2, c3, key0, key1, 10)
        tl.store(out_ptr + offs, a)
        tl.store(out_ptr + N + offs, b)
        tl.store(out_ptr + 2 * N + offs, c)
        tl.store(out_ptr + 3 * N + offs, d)

    N = 32
    rng = np.random.default_rng(2)
    ctr = rng.integers(0, 1 << 32, (4, N), dtype=np.uint64).astype(np.uint32)
    k0, k1 = 0x1234567, 0x7654321            # below 2^31: passed as plain integers
    out = torch.zeros(4 * N, dtype=torch.uint32)
    try:
        block_kernel[(1,)](out, torch.from_numpy(ctr.reshape(-1).copy()), k0, k1, N=N)
    except Exception as exc:                  # the interpreter is not part of what is tested here
        pytest.skip(f"the Triton interpreter could not run the routine: {exc!r}"[:200])
    got = out.numpy().reshape(4, N)
    for j in range(N):
        assert oracle.philox4x32_10(ctr[:, j], [k0, k1]).tolist() == got[:, j].tolist(), j


def test_philox_is_a_bijection_with_good_avalanche(oracle):
    rng = np.random.default_rng(3)
    key = [0xdeadbeef, 0x12345678]
    seen = set()
    for j in range(20000):                                   # consecutive counters, as the operator uses them
        out = tuple(oracle.philox4x32_10([j, 0, 3, 7], key).tolist())
        assert out not in seen
        seen.add(out)
    flips = []
    for _ in range(400):
        ctr = rng.integers(0, 1 << 32, 4).tolist()
        a = oracle.philox4x32_10(ctr, key)
        word, bit = int(rng.integers(0, 4)), int(rng.integers(0, 32))
        ctr[word] ^= 1 << bit
        b = oracle.philox4x32_10(ctr, key)
        flips.append(sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(a, b)))
    assert 60.0 < np.mean(flips) < 68.0                      # 64 of 128 bits, sigma of the mean 0.28
    # bytes of the output are uniform: chi-square over 256 bins, 80000 bytes
    data = np.array([oracle.philox4x32_10([j, 1, 2, 3], key) for j in range(5000)], dtype=np.uint32)
    counts = np.bincount(data.view(np.uint8).ravel(), minlength=256)
    chi2 = float(((counts - counts.mean()) ** 2 / counts.mean()).sum())
    assert chi2 < 350.0                                      # 255 degrees of freedom: mean 255, sigma 22.6


def _definition(u, first_elem, seed, step, worker):
    """The operator as defined, from the big-integer generator."""
    u = np.asarray(u, np.float32)
    s = np.float32(np.max(np.abs(u))) if u.size else np.float32(0)
    q = np.zeros(u.size, np.int32)
    for j, uj in enumerate(u):
        if s == 0:
            continue
        elem = first_elem + j
        words = philox_bigint([(elem >> 2) & M32, (elem >> 2) >> 32, worker, step], [seed & M32, seed >> 32])
        r = np.float32(words[elem & 3] >> 8) * np.float32(2.0 ** -24)
        y = np.float32(abs(uj)) / s
        q[j] = (1 if r < y else 0) * (-1 if uj < 0 else 1)
    return float(s), q


def test_operator_follows_its_definition(oracle):
    rng = np.random.default_rng(4)
    for trial in range(20):
        n = int(rng.integers(1, 60))
        u = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 3)).astype(np.float32)
        if trial % 5 == 0:
            u[rng.integers(0, n)] = 0.0
        first, seed = int(rng.integers(0, 1 << 40)) * 4 + int(rng.integers(0, 4)), int(rng.integers(0, 1 << 63))
        step, worker = int(rng.integers(1, 1 << 20)), int(rng.integers(0, 64))
        s, q, resid = oracle.quantize_grad_segment_stochastic(u, first, seed, step, worker)
        s_def, q_def = _definition(u, first, seed, step, worker)
        assert s == s_def and np.array_equal(q, q_def)
        assert set(np.unique(q)).issubset({-1, 0, 1})
        assert abs(q[np.argmax(np.abs(u))]) == 1              # y = 1: r < 1 always
        assert np.all(q[u == 0] == 0)                         # y = 0: never raised
        assert np.array_equal(resid, u - q.astype(np.float32) * np.float32(s))   # e' = u - Q(u), one rounding
    s, q, resid = oracle.quantize_grad_segment_stochastic(np.zeros(7, np.float32), 0, 1, 1, 0)
    assert s == 0.0 and not q.any() and not resid.any()


def test_operator_is_unbiased(oracle):
    # 16 coordinates, 62 500 steps: a million coins; E Q(u) = u within 4 sigma per coordinate
    u = np.array([1.0, -1.0, 0.5, -0.5, 0.25, 0.75, -0.125, 0.9, 0.01, -0.3, 0.6, 0.05, 0.0, 0.33, -0.66, 0.999],
                 np.float32)
    T = 62500
    total = np.zeros(u.size, np.float64)
    for t in range(1, T + 1):
        _s, q, _r = oracle.quantize_grad_segment_stochastic(u, 128, 20200429, t, 5)
        total += q
    mean = total / T                                          # scale is 1
    p = np.abs(u).astype(np.float64)
    sigma = np.sqrt(np.maximum(p * (1 - p), 1e-12) / T)
    assert np.all(np.abs(mean - u) <= 4 * sigma + 1e-12), (mean - u) / sigma
    # the deterministic ternary quantizer is biased on the same vector (everything below 1/2 is dropped)
    _s, qd, _r = oracle.quantize_grad_segment(u, 0)
    assert np.max(np.abs(qd - u)) >= 0.4


def test_streams_differ_by_worker_step_and_seed(oracle):
    u = np.full(4096, 0.5, np.float32)
    u[0] = 1.0
    base = oracle.quantize_grad_segment_stochastic(u, 0, 1, 1, 0)[1]
    assert 0.45 < np.mean(base[1:] != 0) < 0.55
    for kw in (dict(seed=2), dict(step=2), dict(worker=1), dict(first=4096)):
        other = oracle.quantize_grad_segment_stochastic(u, kw.get("first", 0), kw.get("seed", 1),
                                                        kw.get("step", 1), kw.get("worker", 0))[1]
        agree = np.mean(other[1:] == base[1:])
        assert 0.4 < agree < 0.6, (kw, agree)                 # independent coins agree half the time


@pytest.mark.parametrize("placement", [0, 1])
def test_whole_step_with_the_stochastic_operator(oracle, placement):
    """Through OracleState: the new error buffer is u minus what is sent, codes are ternary
    codes, the scale is max |u|, and the run depends on the seed."""
    rng = np.random.default_rng(6)
    seg, n = [300, 70, 1000], 3
    d = sum(seg)
    runs = []
    for seed in (11, 11, 12):
        st = oracle.OracleState(seg, n, 0, 0, placement, 0.9, 0.999, 1e-8, grid_g=oracle.GRID_STOCHASTIC, seed=seed)
        st.set_weights((np.random.default_rng(7).standard_normal(d) * 0.1).astype(np.float32))
        grng = np.random.default_rng(8)
        for t in range(3):
            g = st.to_padded((grng.standard_normal((n, d)) * 0.01).astype(np.float32))
            e_before = st.e.copy()
            st.workers_step(g, 1e-3)
            for i in range(n):
                codes = oracle.unpack_bits(st.gcodes[i], st.D, 2).astype(np.int32) - 1
                assert set(np.unique(codes)).issubset({-1, 0, 1})
                if placement == 0:
                    u = g[i] + e_before[i]
                    for s, (off, ln) in enumerate(zip(st.seg_off.tolist(), st.seg_len.tolist())):
                        sent = codes[off:off + ln].astype(np.float32) * st.scales[i, s]
                        assert np.array_equal(st.e[i, off:off + ln], u[off:off + ln] - sent)    # e' = fl(u - Q(u))
                        assert st.scales[i, s] == np.max(np.abs(u[off:off + ln]))
            st.server_step(1e-3)
        runs.append((st.x.copy(), st.gcodes.copy()))
    assert np.array_equal(runs[0][1], runs[1][1]) and np.array_equal(runs[0][0], runs[1][0])   # same seed
    assert not np.array_equal(runs[0][1], runs[2][1])                                          # another seed
