"""Pins for the float64 CPU oracle (no GPU needed).

The paper prints no numbers for the plasticity path, so the oracle is pinned to
what the mathematics fixes: hand-derived closed forms (tests/golden), exact
rational arithmetic, a BLAS route, invariants, a negative control, closed-form
and pair-wise brute-force slopes, and hand-replayed Algorithm 1 traces.
"""
from fractions import Fraction
from pathlib import Path

import math
import numpy as np
import pytest
import torch

import oracle
from paper_2201_06227_b200 import workloads as wl

GOLDEN = Path(__file__).parent / "golden"


def bits_of(rows):
    """Exact bf16 bits of a small float matrix (every value must be bf16-exact)."""
    t = torch.tensor(rows, dtype=torch.float32)
    tb = t.to(torch.bfloat16)
    assert torch.equal(tb.to(torch.float32), t), "fixture value is not exact in bfloat16"
    return wl.bf16_bits(tb)


def rand_bits(b, d, seed, relu=False, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn((b, d), generator=g) * scale
    if relu:
        x = torch.relu(x)
    return wl.bf16_bits(x.to(torch.bfloat16))


def as_f64(bits):
    return wl.from_bits(bits).to(torch.float64).numpy()


# ----------------------------------------------------------------------------- closed forms

def _parse_matrix(s):
    return [[float(Fraction(v)) for v in row.split()] for row in s.split(";")]


def _closed_form_cases():
    for line in (GOLDEN / "sp_loss_closed_forms.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        name, b, d, at, ar, exp = [f.strip() for f in line.split("|")]
        yield pytest.param(int(b), int(d), _parse_matrix(at), _parse_matrix(ar), float(exp), id=name)


@pytest.mark.parametrize("b,d,at,ar,expected", list(_closed_form_cases()))
def test_closed_form_fixture(b, d, at, ar, expected):
    A, R = bits_of(at), bits_of(ar)
    assert A.shape == (b, d)
    assert oracle.sp_loss(A, R) == pytest.approx(expected, abs=1e-15)


@pytest.mark.parametrize("seed", range(5))
def test_b2_angle_formula(seed):
    """b = 2: rows of the normalised Gram are unit vectors in the plane, so the loss is
    (1/2)(2 - cos(thetaT - thetaR) - cos(phiT - phiR)) with theta, phi the row angles."""
    A, R = rand_bits(2, 16, seed), rand_bits(2, 16, 100 + seed)

    def angles(bits):
        X = as_f64(bits)
        a, c, e = X[0] @ X[0], X[0] @ X[1], X[1] @ X[1]
        return math.atan2(c, a), math.atan2(e, c)

    tT, pT = angles(A)
    tR, pR = angles(R)
    expected = 0.5 * (2.0 - math.cos(tT - tR) - math.cos(pT - pR))
    assert oracle.sp_loss(A, R) == pytest.approx(expected, rel=1e-12, abs=1e-15)


@pytest.mark.parametrize("b", [2, 3, 4, 9, 16])
def test_onehot_vs_identical_rows(b):
    """Orthogonal rows give G~_T = I, identical rows give G~_R = 1/sqrt(b) everywhere:
    P = (1/b)[(1 - 1/sqrt b)^2 + (b-1)/b]."""
    at = np.eye(b).tolist()
    ar = [[1.0, 2.0, 0.5] + [0.0] * (b - 3 if b > 3 else 0)] * b
    ar = [r[:b] if b >= 3 else r[:b] for r in ar]
    A, R = bits_of(at), bits_of(ar)
    expected = ((1 - 1 / math.sqrt(b)) ** 2 + (b - 1) / b) / b
    assert oracle.sp_loss(A, R) == pytest.approx(expected, rel=1e-13)


# ----------------------------------------------------------------------------- exact arithmetic

@pytest.mark.parametrize("b,d,seed", [(2, 5, 0), (3, 7, 1), (5, 13, 2)])
def test_gram_exact_rationals(b, d, seed):
    """bf16 values are dyadic rationals: the Gram matrix is exact in Fractions."""
    bits = rand_bits(b, d, seed)
    X = as_f64(bits)
    F = [[Fraction(float(v)) for v in row] for row in X]
    G = oracle.gram(bits)
    for i in range(b):
        for j in range(b):
            exact = sum(F[i][k] * F[j][k] for k in range(d))
            assert G[i, j] == pytest.approx(float(exact), rel=1e-14, abs=1e-300)
    # asymmetric index use (a transposed or dropped operand) shows here:
    assert G[0, 1] == pytest.approx(float(sum(F[0][k] * F[1][k] for k in range(d))), rel=1e-14)


def test_gram_not_transposed():
    """A is b x d (samples x features): A A^T is b x b, not d x d."""
    bits = bits_of([[1, 2, 3], [4, 5, 6]])
    G = oracle.gram(bits)
    assert G.shape == (2, 2)
    assert G.tolist() == [[14.0, 32.0], [32.0, 77.0]]


# ----------------------------------------------------------------------------- library route

@pytest.mark.parametrize("b,d,relu", [(8, 4096, True), (17, 72, False), (64, 1000, True), (100, 333, False)])
def test_blas_route(b, d, relu):
    """G is a textbook SYRK; the same steps through numpy's float64 matmul agree."""
    A, R = rand_bits(b, d, 7, relu), rand_bits(b, d, 8, relu)
    loss, gt, gr = oracle.sp_loss(A, R, return_grams=True)

    def route(bits):
        X = as_f64(bits)
        G = X @ X.T
        return G / np.maximum(np.linalg.norm(G, axis=1, keepdims=True), oracle.EPS)

    nt, nr = route(A), route(R)
    np.testing.assert_allclose(gt, nt, rtol=0, atol=1e-13)
    np.testing.assert_allclose(gr, nr, rtol=0, atol=1e-13)
    assert loss == pytest.approx(((nt - nr) ** 2).sum() / b ** 2, rel=1e-10, abs=1e-18)
    # algebraically different route: P = (2/b)(1 - mean_i cos(angle between rows i))
    cosines = (nt * nr).sum(axis=1)
    assert loss == pytest.approx(2.0 / b * (1.0 - cosines.mean()), rel=1e-8, abs=1e-15)


def test_gram_row_matches_gram():
    bits = rand_bits(9, 257, 3)
    G = oracle.gram(bits)
    for i in (0, 4, 8):
        np.testing.assert_allclose(oracle.gram_row(bits, i), G[i], rtol=1e-14)


# ----------------------------------------------------------------------------- invariants

@pytest.mark.parametrize("seed", range(3))
def test_invariants(seed):
    b, d = 12, 96
    A, R = rand_bits(b, d, seed, relu=True), rand_bits(b, d, 50 + seed, relu=True)
    base, gt, gr = oracle.sp_loss(A, R, return_grams=True)
    # identical inputs: exactly zero
    assert oracle.sp_loss(A, A) == 0.0
    # bounds: entries in [-1, 1], unit rows, positive diagonal, 0 <= P <= 2/b for ReLU inputs
    for g in (gt, gr):
        assert np.all(np.abs(g) <= 1 + 1e-15)
        np.testing.assert_allclose(np.linalg.norm(g, axis=1), 1.0, rtol=1e-13)
        assert np.all(np.diag(g) > 0)
    assert 0.0 <= base <= 2.0 / b
    # global scalar on either side (power of two is exact in bf16): unchanged
    A4 = wl.bf16_bits(wl.from_bits(A) * 4.0)
    R8 = wl.bf16_bits(wl.from_bits(R) * 0.125)
    assert oracle.sp_loss(A4, R) == pytest.approx(base, rel=1e-12)
    assert oracle.sp_loss(A, R8) == pytest.approx(base, rel=1e-12)
    # feature permutation (flatten order is immaterial), even a different one per side
    p1 = np.random.default_rng(seed).permutation(d)
    p2 = np.random.default_rng(seed + 9).permutation(d)
    assert oracle.sp_loss(A[:, p1], R[:, p2]) == pytest.approx(base, rel=1e-11)
    # the same sample permutation on both sides
    ps = np.random.default_rng(seed + 5).permutation(b)
    assert oracle.sp_loss(A[ps], R[ps]) == pytest.approx(base, rel=1e-11)
    # symmetric in its two arguments
    assert oracle.sp_loss(R, A) == pytest.approx(base, rel=1e-14)


def test_general_bound_signed_inputs():
    b = 10
    A, R = rand_bits(b, 40, 1), rand_bits(b, 40, 2)
    assert 0.0 <= oracle.sp_loss(A, R) <= 4.0 / b


def test_rotation_invariance():
    """An orthogonal map of the feature axis leaves G, hence P, unchanged.  A signed
    permutation with a Hadamard block keeps every value exact in bf16."""
    b, d = 6, 8
    g = torch.Generator().manual_seed(11)
    X = torch.randint(-4, 5, (b, d), generator=g).to(torch.float32)
    Y = torch.randint(-4, 5, (b, d), generator=g).to(torch.float32)
    H2 = torch.tensor([[1.0, 1.0], [1.0, -1.0]])
    H8 = torch.kron(torch.kron(H2, H2), H2)            # H8 H8^T = 8 I : orthogonal up to a scalar
    base = oracle.sp_loss(bits_of(X.tolist()), bits_of(Y.tolist()))
    rot = oracle.sp_loss(bits_of((X @ H8).tolist()), bits_of((Y @ H8).tolist()))
    assert base > 0
    assert rot == pytest.approx(base, rel=1e-12)


def test_negative_control_row_scaling_changes_loss():
    """Rows of G are normalised, not rows of A: scaling one sample DOES change P.
    (Cosine similarity of the activations would be blind to it.)"""
    A, R = rand_bits(6, 64, 21, relu=True), rand_bits(6, 64, 22, relu=True)
    base = oracle.sp_loss(A, R)
    A2 = A.copy()
    A2[2] = wl.bf16_bits(wl.from_bits(A[2:3]) * 8.0)[0]
    assert abs(oracle.sp_loss(A2, R) - base) > 1e-3 * base


def test_division_is_by_b_squared():
    """P scales as 1/b^2 times the Frobenius sum: duplicating the batch (b -> 2b)
    doubles every squared row norm of G ... checked directly against the sum."""
    A, R = rand_bits(5, 33, 4), rand_bits(5, 33, 5)
    loss, gt, gr = oracle.sp_loss(A, R, return_grams=True)
    assert loss * 25 == pytest.approx(float(((gt - gr) ** 2).sum()), rel=1e-13)


def test_zero_row_clamp():
    A = bits_of([[0, 0, 0], [1, 2, 3]])
    _, gt, _ = oracle.sp_loss(A, A, return_grams=True)
    assert np.all(gt[0] == 0.0)
    assert np.isfinite(gt).all()


# ----------------------------------------------------------------------------- smoothing / slope

def test_smooth_is_mean_of_last_min_window():
    p = np.array([4.0, 2.0, 9.0, 1.0, 5.0, 7.0])
    W = 3
    expect = [4.0, 3.0, 5.0, 4.0, 5.0, 13.0 / 3.0]
    for i, e in enumerate(expect):
        assert oracle.smooth(p, i, W) == pytest.approx(e, rel=1e-15)


@pytest.mark.parametrize("n", [2, 3, 5, 10, 50])
def test_slope_closed_forms(n):
    x = np.arange(n, dtype=np.float64)
    assert oracle.ols_slope(3.0 - 0.25 * x) == pytest.approx(-0.25, rel=1e-13)
    assert oracle.ols_slope(np.full(n, 7.5)) == 0.0
    assert oracle.ols_slope(x * x) == pytest.approx(n - 1, rel=1e-12)   # y = x^2 on 0..n-1


def test_slope_needs_two_points():
    assert oracle.ols_slope(np.array([1.0])) == math.inf


@pytest.mark.parametrize("seed", range(4))
def test_slope_pairwise_brute_force(seed):
    """s = sum_{i<j}(x_j-x_i)(y_j-y_i) / sum_{i<j}(x_j-x_i)^2 (an identity of OLS)."""
    rng = np.random.default_rng(seed)
    n = int(rng.integers(2, 9))
    y = rng.normal(size=n)
    num = sum((j - i) * (y[j] - y[i]) for i in range(n) for j in range(i + 1, n))
    den = sum((j - i) ** 2 for i in range(n) for j in range(i + 1, n))
    assert oracle.ols_slope(y) == pytest.approx(num / den, rel=1e-12, abs=1e-15)
    assert oracle.ols_slope(y) == pytest.approx(np.polyfit(np.arange(n), y, 1)[0], rel=1e-10, abs=1e-13)


def _tok(v):
    if v == "x":
        return None
    if v in ("inf", "-inf"):
        return float(v)
    return float(Fraction(v))


def _trace_cases():
    for line in (GOLDEN / "alg1_traces.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        f = [s.strip() for s in line.split("|")]
        yield pytest.param(int(f[1]), float(f[2]), bool(int(f[3])),
                           [float(v) for v in f[4].split()],
                           [_tok(v) for v in f[5].split()], [_tok(v) for v in f[6].split()],
                           [_tok(v) for v in f[7].split()], int(f[8]), id=f[0])


@pytest.mark.parametrize("W,T,signed,hist,smoothed,slopes,counters,freeze_eval", list(_trace_cases()))
def test_algorithm1_hand_traces(W, T, signed, hist, smoothed, slopes, counters, freeze_eval):
    out = oracle.plasticity_replay(hist, W, T, signed_test=signed)
    assert out["freeze_eval"] == freeze_eval
    assert out["converged"] == (freeze_eval >= 0)
    for i, (sm, sl) in enumerate(zip(smoothed, slopes)):
        if sm is None:
            assert math.isnan(out["smoothed"][i]) and math.isnan(out["slopes"][i])
        else:
            assert out["smoothed"][i] == pytest.approx(sm, rel=1e-6)      # float32 readings
            assert out["slopes"][i] == pytest.approx(sl, rel=1e-6, abs=1e-7)
    # counters: replay prefixes and read the final counter of each
    for i, c in enumerate(counters):
        if c is None:
            continue
        assert oracle.plasticity_replay(hist[: i + 1], W, T, signed_test=signed)["counter"] == c


def test_earliest_convergence_is_W():
    for W in (2, 5, 9):
        out = oracle.plasticity_replay(np.zeros(30, dtype=np.float32), W, 1e-9)
        assert out["freeze_eval"] == W
    # a window of one point has no line to fit: W = 1 never converges
    assert not oracle.plasticity_replay(np.zeros(30, dtype=np.float32), 1, 1.0)["converged"]
    # fewer than W+1 readings can never converge
    assert not oracle.plasticity_replay(np.zeros(5, dtype=np.float32), 5, 1.0)["converged"]


def test_linear_history_slope_after_window_fills():
    """Once the window is full, smoothing a straight line keeps its slope."""
    W, beta = 6, -0.03125
    hist = (2.0 + beta * np.arange(40)).astype(np.float32)
    out = oracle.plasticity_replay(hist, W, 1e-3)
    np.testing.assert_allclose(out["slopes"][2 * W:], beta, rtol=1e-6)
    assert not out["converged"]


def test_nan_is_never_stale():
    hist = np.array([1, 1, np.nan, 1, 1, 1, 1, 1, 1, 1, 1, 1], dtype=np.float32)
    out = oracle.plasticity_replay(hist, 2, 0.5)
    # NaN poisons the smoothed values for W readings and the fit for W more
    assert out["freeze_eval"] > 2 + 2


def test_larger_T_or_smaller_W_freezes_earlier():
    """Sensitivity direction stated in Sec. 6.4: smaller W / larger T freeze earlier."""
    w = wl.WORKLOADS["resnet56"]
    hist = wl.make_history(w, [1e-2] * 4, H=60)[0]
    f = lambda W, T: oracle.plasticity_replay(hist, W, T)["freeze_eval"]
    a, b_, c = f(10, 1e-4), f(10, 1e-3), f(5, 1e-4)
    assert a != -1 and b_ != -1 and b_ < a
    assert c != -1 and c < a
    assert f(10, 1e-12) == -1


# ----------------------------------------------------------------------------- policies around Algorithm 1

def _policy_lines(kind):
    for line in (GOLDEN / "policy_traces.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        if f[0] == kind:
            yield f


def _frac_list(txt):
    out = []
    for tok in txt.split():
        out.append(np.nan if tok == "x" else (np.inf if tok == "inf" else float(Fraction(tok))))
    return np.array(out)


@pytest.mark.parametrize("f", list(_policy_lines("auto")))
def test_auto_tolerance_hand_traces(f):
    W, hist = int(f[1]), np.array([float(v) for v in f[2].split()], dtype=np.float32)
    want = _frac_list(f[3])
    got = oracle.plasticity_replay_auto(hist, W)
    assert got["T"] == pytest.approx(float(Fraction(f[4])), rel=1e-12)
    assert got["freeze_eval"] == int(f[5])
    live = ~np.isnan(want)
    assert np.array_equal(np.isnan(got["slopes"]), ~live)
    fin = live & np.isfinite(want)
    np.testing.assert_allclose(got["slopes"][fin], want[fin], rtol=1e-12, atol=1e-15)
    assert np.all(np.isinf(got["slopes"][live & ~fin]))


def test_auto_tolerance_of_a_straight_line_is_a_tenth_of_its_slope():
    # raw readings a + beta i: the first three smoothed values are a, a + beta/2, a + beta, so both
    # early slopes are beta/2 and T = |beta|/10; once the window is full the slope is beta: never stale
    for beta in (0.3, -2.0):
        hist = (5.0 + beta * np.arange(40)).astype(np.float32)
        got = oracle.plasticity_replay_auto(hist, 6)
        assert got["T"] == pytest.approx(abs(beta) / 10, rel=1e-6)
        assert got["freeze_eval"] == -1
    # a constant history gives T = 0, and |0| < 0 is false: it never freezes either
    got = oracle.plasticity_replay_auto(np.full(30, 2.5, dtype=np.float32), 4)
    assert got["T"] == 0.0 and got["freeze_eval"] == -1


@pytest.mark.parametrize("seed", range(5))
def test_auto_tolerance_equals_fixed_tolerance_after_the_initial_readings(seed):
    # with T known the rule is the plain Algorithm 1, except that evaluations 0..2 cannot be stale:
    # replay with the derived T and compare wherever the fixed-T run was not stale before evaluation 3
    rng = np.random.default_rng(seed)
    k = np.arange(80)
    hist = (np.exp(-k / rng.uniform(3, 15)) + 0.05 + 0.002 * rng.standard_normal(80)).astype(np.float32)
    W = int(rng.integers(3, 8))
    a = oracle.plasticity_replay_auto(hist, W)
    early = [abs(oracle.ols_slope([oracle.smooth(hist, j, W) for j in range(i + 1)][-W:])) for i in (1, 2)]
    assert a["T"] == pytest.approx(0.2 * max(early), rel=1e-12)
    b = oracle.plasticity_replay(hist, W, a["T"])
    stale_early = np.abs(b["slopes"][1:3]) < a["T"]
    if not stale_early.any():
        assert a["freeze_eval"] == b["freeze_eval"]
        np.testing.assert_array_equal(a["slopes"], b["slopes"])


@pytest.mark.parametrize("f", list(_policy_lines("front")))
def test_frontmost_hand_traces(f):
    W = int(f[1])
    T = [float(v) for v in f[2].split()]
    hist = np.array([[float(v) for v in row.split()] for row in f[3].split(";")], dtype=np.float32)
    got = oracle.frontmost_replay(hist, W, T)
    assert got["monitored"].tolist() == [int(v) for v in f[4].split()]
    assert got["freeze_eval"].tolist() == [int(v) for v in f[5].split()]


@pytest.mark.parametrize("seed", range(6))
def test_frontmost_is_single_module_replays_chained(seed):
    # the policy only decides WHICH module is fed: module l's run must be the plain Algorithm 1 on
    # its own readings from the evaluation after module l - 1 froze
    rng = np.random.default_rng(100 + seed)
    M, H, W = 4, 120, int(rng.integers(2, 6))
    k = np.arange(H)
    hist = np.stack([0.3 * np.exp(-k / rng.uniform(2, 10)) + 0.01 * (m + 1) + 1e-4 * rng.standard_normal(H)
                     for m in range(M)]).astype(np.float32)
    T = rng.uniform(2e-3, 2e-2, size=M)
    got = oracle.frontmost_replay(hist, W, T)
    start, frozen = 0, 0
    for m in range(M):
        if start >= H:
            assert got["freeze_eval"][m] == -1
            continue
        single = oracle.plasticity_replay(hist[m, start:], W, float(T[m]))
        if single["converged"]:
            assert got["freeze_eval"][m] == start + single["freeze_eval"]
            n = single["freeze_eval"] + 1
            np.testing.assert_array_equal(got["slopes"][start:start + n], single["slopes"][:n])
            assert np.all(got["monitored"][start:start + n] == m)
            start += n
            frozen += 1
        else:
            assert got["freeze_eval"][m] == -1
            assert np.all(got["monitored"][start:] == m)
            start = H
    assert got["frozen"] == frozen
    fe = got["freeze_eval"]
    assert np.all(fe[:frozen] >= 0) and np.all(fe[frozen:] == -1) and np.all(np.diff(fe[:frozen]) > 0)
    # one module: the policy changes nothing
    one = oracle.frontmost_replay(hist[:1], W, T[:1])
    assert one["freeze_eval"][0] == oracle.plasticity_replay(hist[0], W, float(T[0]))["freeze_eval"]


@pytest.mark.parametrize("f", list(_policy_lines("boot")))
def test_bootstrap_hand_traces(f):
    W, tol = int(f[1]), float(f[2])
    hist = np.array([float(v) for v in f[3].split()], dtype=np.float32)
    want = _frac_list(f[4])
    got = oracle.bootstrap_replay(hist, W, tol)
    assert got["end"] == int(f[5])
    assert np.array_equal(np.isnan(got["rates"]), np.isnan(want))
    np.testing.assert_allclose(got["rates"][~np.isnan(want)], want[~np.isnan(want)], rtol=1e-6)


def test_bootstrap_closed_forms():
    # a constant loss changes by 0 %: the stage ends with the first full window
    assert oracle.bootstrap_replay(np.full(20, 3.0, dtype=np.float32), 5)["end"] == 4
    # a straight line a - beta i: once every smoothed value in the window is a full average
    # (i >= 2W - 2) the fitted slope is -beta and the window mean a - beta (i - W + 1)
    a, beta, W = 100.0, 0.5, 6
    got = oracle.bootstrap_replay((a - beta * np.arange(60)).astype(np.float32), W, 1e-9)
    for i in range(2 * W - 2, 60):
        assert got["rates"][i] == pytest.approx(beta * (W - 1) / (a - beta * (i - W + 1)), rel=1e-6)
    assert got["end"] == -1
    # the rate is relative: scaling the loss by any positive constant changes nothing
    rng = np.random.default_rng(3)
    base = (2.0 * np.exp(-np.arange(50) / 7.0) + 0.3 + 0.01 * rng.random(50)).astype(np.float32)
    r1 = oracle.bootstrap_replay(base, 5, 0.1)
    r2 = oracle.bootstrap_replay(base * np.float32(8.0), 5, 0.1)   # exact in float32
    assert r1["end"] == r2["end"] and r1["end"] > 5
    np.testing.assert_allclose(r1["rates"][4:r1["end"] + 1], r2["rates"][4:r1["end"] + 1], rtol=1e-12)
    # a looser tolerance can only end the stage earlier
    assert oracle.bootstrap_replay(base, 5, 0.3)["end"] <= r1["end"]


# ----------------------------------------------------------------------------- unfreezing on learning-rate annealing

def _unfreeze_lines():
    for line in (GOLDEN / "unfreeze_traces.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        yield [x.strip() for x in line.split("|")]


@pytest.mark.parametrize("f", list(_unfreeze_lines()))
def test_unfreeze_hand_traces(f):
    frontmost, W = bool(int(f[1])), int(f[2])
    T = [float(v) for v in f[3].split()]
    hist = np.array([[float(v) for v in row.split()] for row in f[4].split(";")], dtype=np.float32)
    lr = np.array([float(v) for v in f[5].split()])
    got = oracle.unfreeze_replay(hist, lr, W, T, frontmost=frontmost)
    assert got["window"].tolist() == [int(v) for v in f[6].split()]
    assert ["".join(str(int(v)) for v in row) for row in got["frozen"]] == f[7].split()
    fired = [int(v) for v in f[8].split()]
    assert np.nonzero(got["restarted"])[0].tolist() == fired and got["restarts"] == len(fired)
    want = _frac_list(f[9])
    assert np.array_equal(np.isnan(got["slopes"][0]), np.isnan(want))
    fin = np.isfinite(want)
    np.testing.assert_allclose(got["slopes"][0][fin], want[fin], rtol=1e-6, atol=1e-7)
    assert np.all(np.isinf(got["slopes"][0][~np.isnan(want) & ~fin]))


def _unfreeze_case(seed, M=4, H=160):
    rng = np.random.default_rng(seed)
    k = np.arange(H)
    hist = np.stack([0.3 * np.exp(-(k % 55) / rng.uniform(2, 8)) + 0.01 * (m + 1) + 1e-4 * rng.standard_normal(H)
                     for m in range(M)]).astype(np.float32)
    T = rng.uniform(3e-3, 2e-2, size=M)
    lr = 0.1 * np.power(0.1, k // 55).astype(np.float64)        # step decay by 10x at 55 and 110
    return hist, T, lr


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("frontmost", [False, True])
def test_unfreeze_is_plain_runs_chained(seed, frontmost):
    """Between two restarts the run is the plain rule (already pinned) started afresh on the
    remaining readings with the window in force; the restart is where the learning rate first
    reaches a tenth of its value at the segment's first freeze; the window halves each time."""
    hist, T, lr = _unfreeze_case(seed)
    M, H = hist.shape
    W0 = int(np.random.default_rng(seed).integers(4, 9))
    got = oracle.unfreeze_replay(hist, lr, W0, T, frontmost=frontmost)
    start, W, n_restarts = 0, W0, 0
    while start < H:
        seg = hist[:, start:]
        if frontmost:
            ref = oracle.frontmost_replay(seg, W, T)
            fe = ref["freeze_eval"]
        else:
            runs = [oracle.plasticity_replay(seg[m], W, float(T[m])) for m in range(M)]
            fe = np.array([r["freeze_eval"] for r in runs])
        first = min([e for e in fe if e >= 0], default=None)
        restart_at = None                                       # evaluation of this segment that ends it
        if first is not None:
            later = [i for i in range(first, H - start) if lr[start + i] <= lr[start + first] / 10 * (1 + 1e-6)]
            restart_at = later[0] if later else None
        end = H - start if restart_at is None else restart_at + 1
        assert np.all(got["window"][start:start + end] == W)
        assert got["restarted"][start:start + end].tolist() == [int(i == restart_at) for i in range(end)]
        for i in range(end):
            want = np.zeros(M, dtype=np.uint8) if i == restart_at else ((fe >= 0) & (fe <= i)).astype(np.uint8)
            assert got["frozen"][start + i].tolist() == want.tolist(), (start, i)
        if frontmost:
            for i in range(end):
                for m in range(M):
                    s = got["slopes"][m, start + i]
                    if m == ref["monitored"][i]:
                        assert s == ref["slopes"][i]
                    else:
                        assert np.isnan(s)
        else:
            for m in range(M):
                np.testing.assert_array_equal(got["slopes"][m, start:start + end], runs[m]["slopes"][:end])
        if restart_at is not None:
            n_restarts += 1
            W = max(2, W // 2)
        start += end
    assert got["restarts"] == n_restarts and n_restarts >= 1


def test_unfreeze_needs_a_freeze_and_a_tenfold_drop():
    hist, T, lr = _unfreeze_case(3)
    M, H = hist.shape
    plain = [oracle.plasticity_replay(hist[m], 5, float(T[m])) for m in range(M)]
    # a constant learning rate: nothing ever restarts, the run is the plain rule
    got = oracle.unfreeze_replay(hist, np.full(H, 0.1), 5, T)
    assert got["restarts"] == 0 and np.all(got["window"] == 5)
    for m in range(M):
        np.testing.assert_array_equal(got["slopes"][m], plain[m]["slopes"])
    # a drop by less than ten (x0.2) does not restart either
    got = oracle.unfreeze_replay(hist, np.where(np.arange(H) < 60, 0.1, 0.02), 5, T)
    assert got["restarts"] == 0
    # a tenfold drop BEFORE anything froze is not "since the frontmost freeze": the reference
    # rate is the one at the first freeze, which is already the low one
    first = min(p["freeze_eval"] for p in plain if p["freeze_eval"] >= 0)
    got = oracle.unfreeze_replay(hist, np.where(np.arange(H) < first, 0.1, 0.01), 5, T)
    assert got["restarts"] == 0
    # tolerances that never let anything freeze: no reference rate, no restart
    got = oracle.unfreeze_replay(hist, lr, 5, np.full(M, 1e-12))
    assert got["restarts"] == 0 and not got["frozen"].any()
    # the reference rate is that of the FIRST freeze, not of a later one: module 0 (constant)
    # freezes at 2 under 0.1, module 1 (constant from 4 on) at 6 under 0.05; 0.01 is a tenth of the
    # former only
    two = np.array([[1] * 12, [0, 1, 2, 3, 3, 3, 3, 3, 3, 3, 3, 3]], dtype=np.float32)
    rate = np.array([0.1] * 4 + [0.05] * 4 + [0.01] * 4)
    got = oracle.unfreeze_replay(two, rate, 2, [0.1, 0.1])
    assert got["frozen"][:8].tolist() == [[0, 0]] * 2 + [[1, 0]] * 4 + [[1, 1]] * 2
    assert np.nonzero(got["restarted"])[0].tolist() == [8]
    # a rate that is not positive carries no information
    got = oracle.unfreeze_replay(hist, np.where(np.arange(H) < 60, 0.1, 0.0), 5, T)
    assert got["restarts"] == 0


def test_unfreeze_halves_the_window_with_a_floor_of_two():
    # a constant module freezes W evaluations after each (re)start; the rate falls tenfold every 30
    H = 150
    lr = 0.5 * np.power(0.1, np.arange(H) // 30)
    for W0, want in ((10, [10, 5, 2, 2, 2]), (7, [7, 3, 2, 2, 2]), (3, [3, 2, 2, 2, 2]), (2, [2, 2, 2, 2, 2])):
        got = oracle.unfreeze_replay(np.ones((1, H), dtype=np.float32), lr, W0, [1e-3])
        assert [int(got["window"][30 * k + 15]) for k in range(5)] == want
        assert np.nonzero(got["restarted"])[0].tolist() == [30, 60, 90, 120]
        # frozen W evaluations after the restart (the first evaluation of a run has no line)
        for k in range(5):
            s0 = 0 if k == 0 else 30 * k + 1
            assert got["frozen"][s0 + want[k] - 1, 0] == 0 and got["frozen"][s0 + want[k], 0] == 1


def test_unfreeze_rederives_the_automatic_tolerance():
    # after a restart the initial three readings are those of the new run
    k = np.arange(40)
    run = (np.exp(-k / 4.0) + 0.05).astype(np.float32)
    hist = np.concatenate([run, 3 * run])[None, :]
    lr = np.where(np.arange(80) < 40, 0.1, 0.01)
    got = oracle.unfreeze_replay(hist, lr, 4, None)
    a = oracle.plasticity_replay_auto(run, 4)
    b = oracle.plasticity_replay_auto(3 * run[1:], 2)
    assert a["converged"] and b["converged"]
    assert np.nonzero(got["restarted"])[0].tolist() == [40]
    assert got["frozen"][:, 0].tolist() == ([0] * a["freeze_eval"] + [1] * (40 - a["freeze_eval"]) + [0]
                                            + [0] * b["freeze_eval"] + [1] * (39 - b["freeze_eval"]))
    np.testing.assert_array_equal(got["slopes"][0, 41:], b["slopes"])
