"""Pins for the CPU oracle: each check ties an oracle function to something
the paper or the mathematics fixes (closed forms, invariants, brute force,
library routines on special cases, hand-derived fixtures under tests/golden).
No GPU and no CUDA code is involved here."""
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")
E768 = 768


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


def _bf16_bits(a):
    """float array -> bf16 bit patterns by truncating fp32 values that are
    already exactly representable in bf16 (test inputs are built that way)."""
    a = np.asarray(a, np.float32)
    bits = a.view(np.uint32)
    assert np.all((bits & 0xFFFF) == 0), "test value not representable in bf16"
    return (bits >> 16).astype(np.uint16)


def _round_bf16(a):
    a = np.asarray(a, np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32)


# ------------------------------------------------------------------ logits
def test_logits_one_hot_selects_entries():
    # z[t][e] = sum_h x[t][h] W[e][h]: a one-hot x row picks column h of W_r,
    # a one-hot W row picks x[t][h] (catches transposed operands / wrong strides).
    rng = np.random.default_rng(0)
    T, H, E = 5, 16, 7
    W = _round_bf16(rng.standard_normal((E, H)))
    X = np.zeros((T, H), np.float32)
    hs = [3, 0, 15, 7, 7]
    for t, h in enumerate(hs):
        X[t, h] = 2.0
    z = oracle.router_logits_f64(_bf16_bits(X), _bf16_bits(W))
    for t, h in enumerate(hs):
        np.testing.assert_array_equal(z[t], 2.0 * W[:, h].astype(np.float64))
    X = _round_bf16(rng.standard_normal((T, H)))
    W1 = np.zeros((E, H), np.float32)
    for e in range(E):
        W1[e, (2 * e + 1) % H] = -0.5
    z = oracle.router_logits_f64(_bf16_bits(X), _bf16_bits(W1))
    for e in range(E):
        np.testing.assert_array_equal(z[:, e], -0.5 * X[:, (2 * e + 1) % H].astype(np.float64))


def test_logits_match_library_matmul():
    rng = np.random.default_rng(1)
    T, H, E = 33, 200, 19
    X = _round_bf16(rng.standard_normal((T, H)))
    W = _round_bf16(rng.standard_normal((E, H)) * 0.02)
    z = oracle.router_logits_f64(_bf16_bits(X), _bf16_bits(W))
    ref = X.astype(np.float64) @ W.astype(np.float64).T
    np.testing.assert_allclose(z, ref, rtol=0, atol=1e-12)


def test_logits_small_integers_exact():
    # integer-valued operands: the fp64 sum is exact and equals integer arithmetic
    rng = np.random.default_rng(2)
    X = rng.integers(-8, 9, (9, 64)).astype(np.float32)
    W = rng.integers(-8, 9, (11, 64)).astype(np.float32)
    z = oracle.router_logits_f64(_bf16_bits(X), _bf16_bits(W))
    ref = X.astype(np.int64) @ W.astype(np.int64).T
    np.testing.assert_array_equal(z, ref.astype(np.float64))


# ----------------------------------------------------------------- sigmoid
def test_sigmoid_f64_closed_forms():
    assert oracle.sigmoid_f64(0.0) == 0.5
    for z in [0.1, 1.0, 3.5, 20.0]:
        assert abs(oracle.sigmoid_f64(z) + oracle.sigmoid_f64(-z) - 1.0) < 1e-15
        assert abs(oracle.sigmoid_f64(z) - scipy.special.expit(z)) < 1e-15
    # logit inverse: sigma(log(p/(1-p))) = p
    for p in [0.25, 0.9, 0.01]:
        assert abs(oracle.sigmoid_f64(np.log(p / (1 - p))) - p) < 1e-15


def test_sigmoid_f32_against_real_sigmoid():
    rng = np.random.default_rng(3)
    z = np.concatenate([np.linspace(-30, 30, 2_000_001), rng.uniform(-30, 30, 1_000_000),
                        rng.standard_normal(500_000) * 2]).astype(np.float32)
    s = oracle.sigmoid_f32(z)
    ref = scipy.special.expit(z.astype(np.float64))
    assert np.max(np.abs(s.astype(np.float64) - ref)) <= 2e-7
    assert s.dtype == np.float32


def test_sigmoid_f32_special_values_and_monotone():
    s = oracle.sigmoid_f32(np.array([0.0, -0.0, 100.0, -100.0, 1e30, -1e30, 87.0, -87.0], np.float32))
    assert s[0] == np.float32(0.5) and s[1] == np.float32(0.5)
    assert s[2] == 1.0 and s[4] == 1.0 and s[6] == 1.0
    assert 0.0 < s[3] < 1e-37 and 0.0 < s[5] < 1e-37 and s[5] <= s[3] <= s[7]
    z = np.linspace(-20, 20, 4_000_001).astype(np.float32)
    s = oracle.sigmoid_f32(z)
    assert np.all(np.diff(s) >= 0), "sigmoid_f32 must be non-decreasing"
    # dense sweep over consecutive floats near the top-K score region
    base = np.float32(3.0).view(np.uint32)
    z = (np.arange(200_000, dtype=np.uint32) + base).view(np.float32)
    assert np.all(np.diff(oracle.sigmoid_f32(z)) >= 0)


# ------------------------------------------------------------------- top-K
def _brute_topk(v, K):
    """K passes of arg-max; ties to the lowest index (explicit scan)."""
    v = list(v)
    taken, out = set(), []
    for _ in range(K):
        best = None
        for i, val in enumerate(v):
            if i in taken:
                continue
            if best is None or val > v[best]:
                best = i
        taken.add(best)
        out.append(best)
    return out


@pytest.mark.parametrize("E,K", [(4, 1), (8, 3), (16, 5), (16, 15), (16, 16)])
def test_topk_f64_brute_force_tiny(E, K):
    rng = np.random.default_rng(10 + E + K)
    T = 64
    z = np.round(rng.standard_normal((T, E)) * 2) / 2      # coarse grid: many exact ties
    b = (rng.integers(-2, 3, E) * 0.125).astype(np.float32)
    idx, gate, alpha, gap = oracle.route_f64(z, b, K)
    s = scipy.special.expit(z)
    for t in range(T):
        v = [oracle.sigmoid_f64(z[t, e]) + float(b[e]) for e in range(E)]
        assert list(idx[t]) == _brute_topk(v, K)
        sel = s[t, idx[t]]
        np.testing.assert_allclose(gate[t], sel / sel.sum(), rtol=1e-14)
        vs = sorted(v, reverse=True)
        if K < E:
            assert alpha[t] == vs[K] and gap[t] == vs[K - 1] - vs[K]


@pytest.mark.parametrize("K", [3, 5, 10])
def test_topk_f32_brute_force_with_planted_ties(K):
    rng = np.random.default_rng(20 + K)
    T, E = 48, E768
    z = (rng.standard_normal((T, E)) * 1.5).astype(np.float32)
    # plant exact ties among the largest logits of every token
    for t in range(T):
        top = np.argsort(-z[t])[:4]
        cols = rng.choice(E, 6, replace=False)
        z[t, cols] = z[t, top[rng.integers(0, 4)]]
    b = np.zeros(E, np.float32)
    idx, gate, alpha = oracle.route_f32(z, b, K)
    s = oracle.sigmoid_f32(z)
    for t in range(T):
        v = (s[t] + b).astype(np.float32)
        assert list(idx[t]) == _brute_topk(v, K)
        order = sorted(range(E), key=lambda e: (-v[e], e))
        assert alpha[t] == v[order[K]]
    # gates: fixed left-to-right fp32 sum
    for t in range(T):
        sel = s[t, idx[t]]
        d = np.float32(sel[0])
        for k in range(1, K):
            d = np.float32(d + sel[k])
        np.testing.assert_array_equal(gate[t], (sel / d).astype(np.float32))


def test_topk_constant_bias_shift_keeps_selection():
    # Section 3, centring paragraph: adding one constant to every bias leaves
    # the ranking and the selected set unchanged (binary64 path; shift chosen
    # exactly representable so no rounding interferes with clear gaps).
    rng = np.random.default_rng(30)
    z = rng.standard_normal((200, E768)) * 1.5
    b = (rng.standard_normal(E768) * 0.01).astype(np.float32)
    i0, g0, _, gap = oracle.route_f64(z, b, 10)
    i1, g1, _, _ = oracle.route_f64(z, (b.astype(np.float64) + 0.25).astype(np.float32), 10)
    clear = gap > 1e-6
    assert clear.sum() > 150
    np.testing.assert_array_equal(i0[clear], i1[clear])
    np.testing.assert_allclose(g0[clear], g1[clear], rtol=1e-15)


def test_topk_permuting_experts_permutes_result():
    rng = np.random.default_rng(31)
    z = rng.standard_normal((50, 64))
    b = (rng.standard_normal(64) * 0.05).astype(np.float32)
    perm = rng.permutation(64)
    i0, g0, a0, _ = oracle.route_f64(z, b, 5)
    i1, g1, a1, _ = oracle.route_f64(z[:, perm], b[perm], 5)
    np.testing.assert_array_equal(perm[i1], i0)       # no ties in continuous data
    np.testing.assert_allclose(g1, g0, rtol=1e-15)
    np.testing.assert_array_equal(a0, a1)


def test_gates_ignore_bias_and_sum_to_one():
    # combination weights use the unbiased scores (sentence after Eq. 2)
    z = np.array([[2.0, 1.0, 0.0, -1.0, 3.0, 0.5]])
    b0 = np.zeros(6, np.float32)
    b1 = np.array([0, 0, 0, 0, 0, 0.9], np.float32)   # pushes expert 5 into the set
    i0, g0, _, _ = oracle.route_f64(z, b0, 2)
    i1, g1, _, _ = oracle.route_f64(z, b1, 2)
    assert list(i0[0]) == [4, 0] and list(i1[0]) == [5, 4]
    s = scipy.special.expit(z[0])
    np.testing.assert_allclose(g0[0], [s[4] / (s[4] + s[0]), s[0] / (s[4] + s[0])], rtol=1e-15)
    np.testing.assert_allclose(g1[0], [s[5] / (s[5] + s[4]), s[4] / (s[5] + s[4])], rtol=1e-15)
    assert abs(g0.sum() - 1) < 1e-15 and abs(g1.sum() - 1) < 1e-15
    # K equal scores -> 1/K each, fp32 chain
    zz = np.full((1, 8), 0.7, np.float32)
    _, g, _ = oracle.route_f32(zz, np.zeros(8, np.float32), 4)
    np.testing.assert_array_equal(g[0], np.full(4, 0.25, np.float32))


def test_route_f32_agrees_with_f64_when_gap_is_clear():
    rng = np.random.default_rng(32)
    z = (rng.standard_normal((300, E768)) * 1.5).astype(np.float32)
    b = (rng.standard_normal(E768) * 0.02).astype(np.float32)
    i64, g64, a64, gap = oracle.route_f64(z.astype(np.float64), b, 10)
    i32, g32, a32 = oracle.route_f32(z, b, 10)
    clear = gap > 1e-5
    assert clear.sum() > 250
    assert np.array_equal(np.sort(i64[clear], 1), np.sort(i32[clear], 1))
    same_order = np.all(i64 == i32, axis=1)
    np.testing.assert_allclose(g32[same_order], g64[same_order], atol=3e-7)
    np.testing.assert_allclose(a32, a64, atol=4e-7)


# ------------------------------------------------------------------- loads
def test_loads_sum_and_recount():
    rng = np.random.default_rng(40)
    T, K = 500, 10
    idx = np.stack([rng.choice(E768, K, replace=False) for _ in range(T)]).astype(np.int32)
    n = oracle.load_counts(idx, E768)
    assert n.sum() == T * K and n.max() <= T           # every token gives exactly K counts
    np.testing.assert_array_equal(n, np.bincount(idx.ravel(), minlength=E768))
    n2 = oracle.load_counts(idx, E768, n.copy())       # microbatches accumulate
    np.testing.assert_array_equal(n2, 2 * n)
    with pytest.raises(ValueError):
        oracle.load_counts(np.array([[E768]], np.int32), E768)


# ------------------------------------------------------------------- error
def test_error_properties():
    rng = np.random.default_rng(41)
    n = rng.integers(0, 400, E768).astype(np.int64)
    n[5] = 0
    e = oracle.load_error(n)
    nbar = n.sum() / E768
    np.testing.assert_allclose(e, (nbar - n) / nbar, rtol=1e-7)
    assert abs(e.astype(np.float64).sum()) < E768 * 1e-7   # sum_i e_i = 0 (Section 3)
    assert e[5] == 1.0                                      # empty expert: e = 1
    assert np.all(oracle.load_error(np.full(E768, 37, np.int64)) == 0)
    assert np.all(e[n > nbar] < 0) and np.all(e[n < nbar] > 0)   # sign convention
    with pytest.raises(ValueError):
        oracle.load_error(np.zeros(E768, np.int64))


# ------------------------------------------------------------- controllers
def _frac(s):
    return float(Fraction(s))


def _half_loads(a, b_):
    n = np.empty(E768, np.int64)
    n[:384], n[384:] = a, b_
    return n


@pytest.mark.parametrize("row", _rows("id_trajectories.txt"))
def test_id_closed_form_trajectories(row):
    case, steps, bA, bB = row[0], int(row[1]), _frac(row[2]), _frac(row[3])
    ki = kd = 2.0 ** -7
    b = np.zeros(E768, np.float32)
    ep = np.zeros(E768, np.float32)
    for t in range(steps):
        n = _half_loads(512, 1536) if case == "const" else _half_loads(1024 - 16 * (t + 1), 1024 + 16 * (t + 1))
        e = oracle.load_error(n)
        b, ep, g = oracle.id_update(b, ep, e, ki, kd, center=True)
        expect_gate = 1 if (case == "grow" and t >= 1) else 0
        assert np.all(g == expect_gate)
    assert np.all(b[:384] == np.float32(bA)) and np.all(b[384:] == np.float32(bB))


@pytest.mark.parametrize("row", _rows("gate_truth_table.txt"))
def test_id_gate_truth_table(row):
    e_prev, e, gate = np.float32(row[0]), np.float32(row[1]), int(row[2])
    b0 = np.zeros(4, np.float32)
    ki, kd = np.float32(0.5), np.float32(0.25)
    b, ep, g = oracle.id_update(b0, np.full(4, e_prev), np.full(4, e), ki, kd, center=False)
    assert np.all(g == gate)
    de = np.float32(e - e_prev)
    expect = np.float32(np.float32(ki * e) + (np.float32(kd * de) if gate else np.float32(0)))
    assert np.all(b == expect) and np.all(ep == e)


def test_id_integral_only_reduces_to_eq9_and_keeps_zero_mean():
    # Kd = 0: b(t+1) = b(t) + Ki e(t) (Eq. 9); sum_i e_i = 0 keeps the mean
    # at zero so centring changes (almost) nothing.
    rng = np.random.default_rng(50)
    b = np.zeros(E768, np.float32)
    bc = np.zeros(E768, np.float32)
    ep = np.zeros(E768, np.float32)
    epc = ep.copy()
    acc = np.zeros(E768, np.float64)
    for t in range(30):
        n = rng.integers(0, 300, E768).astype(np.int64)
        e = oracle.load_error(n)
        b, ep, g = oracle.id_update(b, ep, e, 6e-3, 0.0, center=False)
        bc, epc, _ = oracle.id_update(bc, epc, e, 6e-3, 0.0, center=True)
        acc += 6e-3 * e.astype(np.float64)
        assert True  # gate value is irrelevant when Kd = 0
    np.testing.assert_allclose(b, acc, atol=2e-6)
    assert abs(b.astype(np.float64).mean()) < 1e-7
    np.testing.assert_allclose(bc, b, atol=3e-7)


def test_id_derivative_inactive_while_imbalance_shrinks():
    # errors shrink monotonically without changing sign: gate stays closed, so
    # Kd has no effect (Section 3: closed when the error moves toward zero).
    b0 = np.zeros(E768, np.float32)
    b1 = np.zeros(E768, np.float32)
    ep0 = np.zeros(E768, np.float32)
    ep1 = np.zeros(E768, np.float32)
    for t in range(12):
        d = 600 - 40 * t
        e = oracle.load_error(_half_loads(1024 - d, 1024 + d))
        b0, ep0, g0 = oracle.id_update(b0, ep0, e, 6e-3, 0.0)
        b1, ep1, g1 = oracle.id_update(b1, ep1, e, 6e-3, 6e-3)
        assert not g1.any()
    np.testing.assert_array_equal(b0, b1)


def test_id_general_step_against_fp64_formula_and_centering():
    rng = np.random.default_rng(51)
    b = (rng.standard_normal(E768) * 0.01).astype(np.float32)
    ep = (rng.standard_normal(E768) * 0.5).astype(np.float32)
    e = oracle.load_error(rng.integers(0, 300, E768).astype(np.int64))
    ki, kd = 6e-3, 6e-3
    bn, epn, g = oracle.id_update(b, ep, e, ki, kd, center=True)
    de = e.astype(np.float64) - ep
    gate = (ep.astype(np.float64) * de) > 0
    np.testing.assert_array_equal(g.astype(bool), gate)
    assert 0 < gate.sum() < E768
    bt = b + ki * e.astype(np.float64) + kd * gate * de          # Eq. 12, first line
    ref = bt - bt.mean()                                          # Eq. 12, second line
    np.testing.assert_allclose(bn, ref, atol=2e-7)
    assert abs(bn.astype(np.float64).sum()) < E768 * 6e-8         # sum_i b_i = 0
    np.testing.assert_array_equal(epn, e)
    # centring alone: mean within one ulp of the sequential fp64 mean
    c = oracle.center(b)
    np.testing.assert_allclose(c, b - np.float32(b.astype(np.float64).mean()), atol=1e-9)


def test_fixed_step_is_eta_times_sum_of_signs():
    # Eq. 5: b(t) = eta * sum_tau sign(e(tau)); zero error gives no step
    rng = np.random.default_rng(52)
    eta = 2.0 ** -10
    b = np.zeros(E768, np.float32)
    ep = np.zeros(E768, np.float32)
    signs = np.zeros(E768, np.int64)
    for t in range(25):
        n = rng.integers(0, 5, E768).astype(np.int64)
        n[-1] += (-n.sum()) % E768          # make nbar an integer so that e == 0 occurs
        e = oracle.load_error(n)
        assert (e == 0).any()
        b, ep = oracle.fixed_step_update(b, ep, e, eta)
        signs += np.sign(e).astype(np.int64)
    np.testing.assert_array_equal(b, (signs * eta).astype(np.float32))
    # constant loads: b = t * eta * sign(e)
    b = np.zeros(E768, np.float32)
    for t in range(7):
        b, _ = oracle.fixed_step_update(b, ep, oracle.load_error(_half_loads(10, 30)), eta)
    assert np.all(b[:384] == 7 * eta) and np.all(b[384:] == -7 * eta)


# ---------------------------------------------------------------------- QB
def test_quantile_target_places_q_tokens_above_cutoff():
    # Section 2.3: with cutoffs alpha_i held fixed, the target puts about
    # q = m K / E biased margins above zero per expert (exactly floor(q) with
    # distinct margins under the nearest-rank reading).
    rng = np.random.default_rng(60)
    m, E, K = 512, 64, 4
    z = (rng.standard_normal((m, E)) * 1.5).astype(np.float32)
    b = (rng.standard_normal(E) * 0.05).astype(np.float32)
    _, _, alpha = oracle.route_f32(z, b, K)
    Q = oracle.quantile_target(z, alpha, K)
    S = oracle.sigmoid_f32(z)
    margin = S - alpha[:, None]
    r = m - (m * K) // E
    np.testing.assert_array_equal(Q, -np.sort(margin, axis=0)[r - 1])      # position vs a full sort
    q = (m * K) // E
    above = (margin > -Q[None, :]).sum(axis=0)
    at_or_above = (margin >= -Q[None, :]).sum(axis=0)
    assert np.all(above <= q) and np.all(at_or_above >= q + 1)
    distinct = (margin == -Q[None, :]).sum(axis=0) == 1          # no tie at the cutoff
    assert distinct.sum() > E // 2 and np.all(above[distinct] == q)
    # rho = 0 stores the target; EMA blends
    e = np.zeros(E, np.float32)
    b0, _ = oracle.quantile_update(b, e, e, Q, rho=0.0)
    np.testing.assert_array_equal(b0, Q)
    b5, _ = oracle.quantile_update(b, e, e, Q, rho=0.5)
    np.testing.assert_allclose(b5, 0.5 * b + 0.5 * Q, atol=1e-8)


def test_quantile_histogram_estimate_hand_example():
    # logits 0 give the score 0.5 exactly, so alpha_i = 0.5 - d_i plants the margins d = -0.5, -0.25, 0.25, 0.5.
    # B = 4 bins over [-1, 1): edges -1, -0.5, 0, 0.5, 1 -> counts [0, 2, 1, 1].  E = 4, K = 1: r = 4 - 1 = 3,
    # the third smallest margin (0.25) sits alone in bin 2 (below = 2, count = 1): est = -1 + (2 + 0.5) * 0.5
    # = 0.25, Q = -0.25.  With K = 2: r = 2, bin 1 (below = 0, count = 2): est = -1 + (1 + 1.5 / 2) * 0.5 = -0.125.
    d = np.array([-0.5, -0.25, 0.25, 0.5], np.float32)
    z = np.zeros((4, 4), np.float32)
    alpha = (np.float32(0.5) - d).astype(np.float32)
    Q, hist = oracle.quantile_target_hist(z, alpha, 1, 4, 1.0, return_hist=True)
    np.testing.assert_array_equal(hist, np.tile(np.array([0, 2, 1, 1]), (4, 1)))
    np.testing.assert_array_equal(Q, np.full(4, -0.25, np.float32))
    np.testing.assert_array_equal(oracle.quantile_target_hist(z, alpha, 2, 4, 1.0), np.full(4, 0.125, np.float32))
    # margins outside the range count in the end bins: range 0.375 -> bins of width 0.1875 over [-0.375, 0.375)
    _, hist = oracle.quantile_target_hist(z, alpha, 1, 4, 0.375, return_hist=True)
    np.testing.assert_array_equal(hist[0], np.array([2, 0, 0, 2]))


@pytest.mark.parametrize("bins,value_range", [(64, 1.0), (1024, 1.0), (4096, 2.0), (512, 0.25)])
def test_quantile_histogram_estimate_is_within_one_bin_of_the_exact_target(bins, value_range):
    # the exact r-th smallest margin lies in the bin the estimate interpolates in: |estimate - exact| < bin width
    # wherever the exact value is inside the range; counts of every expert sum to m; finer bins converge
    rng = np.random.default_rng(61)
    m, E, K = 700, 48, 5
    z = (rng.standard_normal((m, E)) * 1.5).astype(np.float32)
    b = (rng.standard_normal(E) * 0.05).astype(np.float32)
    _, _, alpha = oracle.route_f32(z, b, K)
    exact = oracle.quantile_target(z, alpha, K)
    est, hist = oracle.quantile_target_hist(z, alpha, K, bins, value_range, return_hist=True)
    assert np.all(hist.sum(axis=1) == m)
    h = 2.0 * value_range / bins
    inside = np.abs(exact) < value_range - h
    assert inside.sum() >= E // 2
    assert np.max(np.abs(est[inside].astype(np.float64) - exact[inside])) < h * (1 + 1e-6)
    # histogram = direct binning of the margins (numpy in binary32, same two rounded operations)
    margin = oracle.sigmoid_f32(z) - alpha[:, None]
    u = (margin + np.float32(value_range)) * (np.float32(bins) / (np.float32(2.0) * np.float32(value_range)))
    k = np.clip(np.floor(u), 0, bins - 1).astype(np.int64)
    for j in (0, E // 2, E - 1):
        np.testing.assert_array_equal(hist[j], np.bincount(k[:, j], minlength=bins))


def test_quantile_histogram_estimate_converges_to_the_exact_target():
    rng = np.random.default_rng(62)
    m, E, K = 300, 16, 2
    z = (rng.standard_normal((m, E))).astype(np.float32)
    _, _, alpha = oracle.route_f32(z, np.zeros(E, np.float32), K)
    exact = oracle.quantile_target(z, alpha, K).astype(np.float64)
    errs = [np.max(np.abs(oracle.quantile_target_hist(z, alpha, K, B, 1.0).astype(np.float64) - exact))
            for B in (16, 256, 4096, 65536, 1 << 20)]
    assert all(e < 2.0 / B * 1.000001 for e, B in zip(errs, (16, 256, 4096, 65536, 1 << 20)))
    assert errs[-1] < 2e-6 and errs[-1] < errs[0]


# ----------------------------------------------------------------- metrics
@pytest.mark.parametrize("row", _rows("violation_bounds.txt"))
def test_violation_bounds(row):
    E, K, bound = int(row[0]), int(row[1]), float(row[2])
    T = 1000
    n = np.zeros(E, np.int64)
    n[:K] = T                                      # every token picks the same K experts
    mx, mn = oracle.violations(n)
    assert abs(mx - bound) < 1e-4 and mn == 1.0
    rng = np.random.default_rng(E + K)
    idx = np.stack([rng.choice(E, K, replace=False) for _ in range(200)]).astype(np.int32)
    n = oracle.load_counts(idx, E)
    mx, mn = oracle.violations(n)
    assert 0 <= mx <= bound + 1e-6 and 0 <= mn <= 1
    assert (mn == 1.0) == bool((n == 0).any())
    nbar = n.sum() / E
    np.testing.assert_allclose([mx, mn], [(n.max() - nbar) / nbar, (nbar - n.min()) / nbar], rtol=1e-7)
    mx, mn = oracle.violations(np.full(E, 13, np.int64))
    assert mx == 0 and mn == 0


# ------------------------------------------------------------- diagnostics
def test_load_diagnostics_closed_forms():
    E = 768
    # perfectly balanced: busiest 10 % of the experts (77 of 768) hold 77/768 of the assignments (target 0.10)
    n = np.full(E, 40, np.int64)
    z = np.zeros(E, np.float32)
    g = np.zeros(E, np.int32)
    d = oracle.load_diagnostics(n, g, z, z)
    assert abs(d[1] - 77 / 768) < 1e-7 and d[0] == 0 and d[2] == 0 and d[3] == 0
    # everything on 3 experts: share 1, inactive ratio (E-3)/E
    n = np.zeros(E, np.int64)
    n[[5, 100, 700]] = [10, 20, 30]
    g[:192] = 1
    b0 = np.zeros(E, np.float32)
    b1 = np.full(E, 0.25, np.float32)
    b1[::2] = -0.25
    d = oracle.load_diagnostics(n, g, b0, b1)
    assert d[1] == 1.0 and abs(d[2] - 765 / 768) < 1e-7 and d[0] == np.float32(0.25) and d[3] == np.float32(0.25)
    # share against an explicit partial sort
    rng = np.random.default_rng(70)
    n = rng.integers(0, 500, E).astype(np.int64)
    d = oracle.load_diagnostics(n, g, b0, b0)
    np.testing.assert_allclose(d[1], np.sort(n)[::-1][:77].sum() / n.sum(), rtol=1e-7)
    assert oracle.load_diagnostics(np.arange(1, 11, dtype=np.int64), np.zeros(10, np.int32), z[:10], z[:10])[1] == np.float32(10 / 55)


def test_gate_entropy_closed_forms():
    # uniform weights over K experts: H = ln K; a one-hot weight vector: H = 0
    for K in (3, 8, 10):
        w = np.full((7, K), 1.0 / K, np.float32)
        assert abs(oracle.gate_entropy_mean(w) - np.log(K)) < 1e-6
    w = np.zeros((4, 5), np.float32)
    w[:, 2] = 1.0
    assert oracle.gate_entropy_mean(w) == 0.0
    rng = np.random.default_rng(71)
    w = rng.random((50, 10)).astype(np.float32)
    w /= w.sum(1, keepdims=True)
    ref = scipy.special.entr(w.astype(np.float64)).sum(1).mean()
    assert abs(oracle.gate_entropy_mean(w) - ref) < 1e-12


def test_full_pool_entropy_closed_forms_and_library():
    E = 768
    # equal logits, zero bias: both score families are uniform over the pool, H = ln E
    z = np.full((5, E), 0.7, np.float32)
    for kind in ("biased_sigmoid", "softmax"):
        assert abs(oracle.full_pool_entropy_mean(z, None, kind) - np.log(E)) < 1e-12
    # softmax entropy ignores a common shift of the logits; it never exceeds ln E
    rng = np.random.default_rng(72)
    z = rng.normal(0, 2.0, (40, E)).astype(np.float32)
    h = oracle.full_pool_entropy_mean(z, None, "softmax")
    zs = (z.astype(np.float64) + 3.0).astype(np.float32)   # shift representable up to fp32 rounding of z
    assert abs(oracle.full_pool_entropy_mean(zs, None, "softmax") - h) < 1e-5
    assert 0.0 < h < np.log(E)
    # against the library softmax / entropy routines
    p = scipy.special.softmax(z.astype(np.float64), axis=1)
    assert abs(h - scipy.special.entr(p).sum(1).mean()) < 1e-12
    b = rng.normal(0, 0.05, E).astype(np.float32)
    c = np.maximum(scipy.special.expit(z.astype(np.float64)) + b.astype(np.float64), 0.0)
    q = c / c.sum(1, keepdims=True)
    assert abs(oracle.full_pool_entropy_mean(z, b, "biased_sigmoid") - scipy.special.entr(q).sum(1).mean()) < 1e-12
    # the bias enters the biased-sigmoid family and not the softmax family
    assert oracle.full_pool_entropy_mean(z, b, "softmax") == h
    assert oracle.full_pool_entropy_mean(z, b, "biased_sigmoid") != oracle.full_pool_entropy_mean(z, None, "biased_sigmoid")
    # clamping: experts whose biased score is negative leave the pool; the remaining n equal scores give ln n
    z = np.zeros((3, E), np.float32)
    b = np.zeros(E, np.float32)
    b[100:] = -0.75                      # 0.5 - 0.75 < 0 -> clamped to zero
    assert abs(oracle.full_pool_entropy_mean(z, b, "biased_sigmoid") - np.log(100)) < 1e-12
    b[:] = -0.75                         # nothing left: no distribution, H = 0
    assert oracle.full_pool_entropy_mean(z, b, "biased_sigmoid") == 0.0
    # two-level distribution: one expert with weight a, the others sharing 1 - a
    z = np.zeros((1, 8), np.float32)
    z[0, 0] = np.log(7.0)                # softmax: p0 = 7/14 = 1/2, others 1/14 each
    want = 0.5 * np.log(2.0) + 0.5 * np.log(14.0)
    assert abs(oracle.full_pool_entropy_mean(z, None, "softmax") - want) < 1e-7


def test_aux_loss_statistics_closed_forms():
    E, T, K = 64, 208, 4
    rng = np.random.default_rng(73)
    z = rng.normal(0, 1.5, (T, E)).astype(np.float32)
    # perfectly even loads: f_i = K/E for all i, and sum_i P_i = 1, so sum_i f_i P_i = K/E whatever the router says
    assert (T * K) % E == 0
    n = np.full(E, (T * K) // E, np.int64)
    f, P, aux = oracle.aux_loss_stats(z, n)
    assert abs(P.sum() - 1.0) < 1e-12 and abs(f.sum() - K) < 1e-12
    np.testing.assert_allclose(P, scipy.special.softmax(z.astype(np.float64), axis=1).mean(0), rtol=1e-12)
    assert abs(aux - K / E) < 1e-12
    np.testing.assert_allclose(aux, float((f * P).sum()), rtol=1e-13)
    # all tokens sent to experts 0..K-1 by a router that is certain of expert 0: f_0 = 1, P_0 ~ 1, aux ~ 1
    z = np.full((T, E), -30.0, np.float32)
    z[:, 0] = 30.0
    n = np.zeros(E, np.int64)
    n[:K] = T
    f, P, aux = oracle.aux_loss_stats(z, n)
    assert f[0] == 1.0 and abs(P[0] - 1.0) < 1e-12 and abs(aux - 1.0) < 1e-12
    # uniform router, any loads: P_i = 1/E, aux = (1/E) sum_i f_i = K/E
    z = np.zeros((T, E), np.float32)
    n = rng.multinomial(T * K, np.ones(E) / E).astype(np.int64)
    f, P, aux = oracle.aux_loss_stats(z, n)
    np.testing.assert_allclose(P, 1.0 / E, rtol=1e-13)
    assert abs(aux - K / E) < 1e-12
    # the loss grows when load and probability concentrate on the same experts (what Eq. 8 penalises)
    z = rng.normal(0, 1.0, (T, E)).astype(np.float32)
    z[:, :4] += 3.0
    hot = np.zeros(E, np.int64); hot[:4] = T
    cold = np.zeros(E, np.int64); cold[-4:] = T
    assert oracle.aux_loss_stats(z, hot)[2] > oracle.aux_loss_stats(z, cold)[2]


# ------------------------------------------------------------- whole chain
def test_route_tokens_chain_and_threads_agree():
    from paper_2609_39137_b200 import synth
    wl = synth.WORKLOADS["tiny_top3"].with_(T=96)
    x = synth.bf16_bits(synth.hidden_states(wl, 0, 0))
    w = synth.bf16_bits(synth.router_weights(wl, 0))
    b = np.zeros(wl.E, np.float32)
    r1 = oracle.route_tokens_f64(x, w, b, wl.K, threads=1)
    r3 = oracle.route_tokens_f64(x, w, b, wl.K, threads=3)
    for k in ("z", "idx", "gate", "alpha", "gap", "n"):
        np.testing.assert_array_equal(r1[k], r3[k])
    assert r1["n"].sum() == 96 * wl.K
    np.testing.assert_array_equal(r1["n"], np.bincount(r1["idx"].ravel(), minlength=wl.E))
