"""Pins for the mask-rule half of the CPU oracle (window map -> true mask -> patterns -> extension).

None of these tests re-types the oracle's formula and compares it with itself: each one checks the
oracle against something the paper prints, a closed form, an invariant, or a brute force built from
the literal pattern matrices of Sec. 4.2.4.
"""
import math
import os

import numpy as np
import pytest

from oracle import dam_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_table2():
    out = {}
    with open(os.path.join(GOLDEN, "table2_boxcox.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


# ---- Table 2 / Sec. 4.2.2 -------------------------------------------------------------------------
@pytest.mark.parametrize("eps_key", ["eps_main", "eps_appendix"])
def test_boxcox_extremes_match_table2(eps_key):
    g = _golden_table2()
    eps = g[eps_key]
    a = orc.amplify_f64(np.array([1.0, 0.0, eps, eps / 10]), g["lambda"], eps)
    # a probability of 1 maps to the table's maximum (printed with two decimals)
    assert f"{a[0]:.2f}" == f"{g['max_value']:.2f}"
    assert a[0] < 2.0                       # 2 - 2*sqrt(eps), strictly below 2
    assert abs(a[0] - (2.0 - 2.0 * math.sqrt(eps))) < 1e-12
    # cells whose map value is 0 (or below eps) are exactly 0 after the shift: the table's zero entries
    assert a[1] == 0.0 and a[2] == 0.0 and a[3] == 0.0


def test_min_over_a_full_map_is_the_constant():
    """The shift subtracts the minimum over all cells; a causal map has zeros above the diagonal, so the
    literal minimum over one amplified map is 0 after the shift, i.e. the shift constant is B(eps)."""
    rng = np.random.default_rng(0)
    L, d = 24, 8
    Q = rng.standard_normal((L, d)).astype(np.float32)
    K = rng.standard_normal((L, d)).astype(np.float32)
    P = orc.window_probs(Q, K, L, 1 / math.sqrt(d))
    a = orc.amplify_f64(P, 0.5, 1e-8)
    assert a.min() == 0.0
    assert np.all(a[np.triu_indices(L, 1)] == 0.0)
    assert np.all(a[np.tril_indices(L)] > 0.0)
    # amplification is monotone: order of cells is preserved
    lo = np.tril_indices(L)
    assert np.array_equal(np.argsort(P[lo], kind="stable"), np.argsort(a[lo], kind="stable"))


def test_log_branch_lambda_zero():
    a = orc.amplify_f64(np.array([1.0, math.e ** -2]), 0.0, 1e-8)
    assert abs(a[0] - (-math.log(1e-8))) < 1e-9
    assert abs(a[0] - a[1] - 2.0) < 1e-9


# ---- window map ---------------------------------------------------------------------------------------
def test_window_probs_rows_sum_to_one_and_causal():
    rng = np.random.default_rng(1)
    L, d = 40, 16
    Q = rng.standard_normal((L, d)).astype(np.float32)
    K = rng.standard_normal((L, d)).astype(np.float32)
    P = orc.window_probs(Q, K, L, 1 / math.sqrt(d))
    assert np.allclose(P.sum(1), 1.0, atol=1e-12)
    assert np.all(P[np.triu_indices(L, 1)] == 0.0)
    assert P[0, 0] == 1.0
    # brute force with numpy on the same inputs
    S = (Q.astype(np.float64) @ K.astype(np.float64).T) / math.sqrt(d)
    S[np.triu_indices(L, 1)] = -np.inf
    E = np.exp(S - S.max(1, keepdims=True))
    assert np.allclose(P, E / E.sum(1, keepdims=True), atol=1e-14)


def test_window_uses_strided_heads():
    """Q [T, H, d] views: the head stride must be honoured (a transposed / wrong-stride read fails)."""
    rng = np.random.default_rng(2)
    T, H, d = 12, 3, 8
    Q = rng.standard_normal((T, H, d)).astype(np.float32)
    K = rng.standard_normal((T, H, d)).astype(np.float32)
    for h in range(H):
        P = orc.window_probs(Q[:, h, :], K[:, h, :], T, 0.3)
        P2 = orc.window_probs(np.ascontiguousarray(Q[:, h, :]), np.ascontiguousarray(K[:, h, :]), T, 0.3)
        assert np.array_equal(P, P2)


# ---- threshold ----------------------------------------------------------------------------------------
def test_threshold_flip_point_close_to_closed_form():
    """m = [2(sqrt(max(p,eps)) - sqrt(eps)) >= tau]  <=>  p >= (tau/2 + sqrt(eps))^2."""
    eps = 1e-8
    for tau in (0.3, 0.1, 0.05, 0.02):
        pstar = (tau / 2 + math.sqrt(eps)) ** 2
        ps = np.array([[pstar * (1 - 1e-5), pstar * (1 + 1e-5)], [0.0, 1.0]])
        M = orc.true_mask_f64(ps, tau, 0.5, eps)
        assert M.tolist() == [[0, 1], [0, 1]]
        M32 = orc.true_mask_f32(ps.astype(np.float32), np.float32(tau), np.float32(eps))
        assert M32.tolist() == [[0, 1], [0, 1]]


def test_threshold_f32_is_monotone_with_single_flip():
    """The single-precision chain is a step function of p: scanning consecutive floats around the flip
    point shows exactly one 0 -> 1 transition."""
    tau, eps = np.float32(0.3), np.float32(1e-8)
    centre = np.float32((0.15 + 1e-4) ** 2)
    bits = centre.view(np.uint32).astype(np.int64) + np.arange(-2048, 2048)
    ps = bits.astype(np.uint32).view(np.float32).reshape(64, 64)
    M = orc.true_mask_f32(np.ascontiguousarray(ps), tau, eps).reshape(-1)
    assert M[0] == 0 and M[-1] == 1
    assert np.count_nonzero(np.diff(M.astype(np.int8))) == 1


def test_capacity_bound_per_row():
    """Probabilities sum to 1, so a row keeps at most floor(1/p*) keys: 44 at the paper's tau = 0.3."""
    rng = np.random.default_rng(3)
    L, d = 200, 4
    Q = (0.05 * rng.standard_normal((L, d))).astype(np.float32)
    K = (0.05 * rng.standard_normal((L, d))).astype(np.float32)
    P = orc.window_probs(Q, K, L, 1.0)
    M = orc.true_mask_f64(P, 0.3, 0.5, 1e-8)
    assert M.sum(1).max() <= 44
    assert M.sum(1).max() >= 40          # near-uniform rows come close to the bound
    assert M[0, 0] == 1                  # row 0 has p = 1
    assert np.all(M[np.triu_indices(L, 1)] == 0)


def test_uniform_attention_closed_form():
    """Q = 0 gives p_ij = 1/(i+1).  At tau = 0.3 rows 0..43 are full (1/44 >= p*), later rows are empty;
    counts are max(0, 44 - k) for both diagonals and columns."""
    L, d = 96, 8
    Q = np.zeros((L, d), np.float32)
    K = np.random.default_rng(4).standard_normal((L, d)).astype(np.float32)
    P = orc.window_probs(Q, K, L, 1 / math.sqrt(d))
    hm = orc.head_mask_from_probs(P, S=300, tau=0.3, mu=0.8)
    for i in range(L):
        expect = np.zeros(L, np.uint8)
        if i + 1 <= 44:
            expect[: i + 1] = 1
        assert np.array_equal(hm.M[i], expect), i
    k = np.arange(L)
    assert np.array_equal(hm.cntD, np.maximum(0, 44 - k))
    assert np.array_equal(hm.cntV, np.maximum(0, 44 - k))
    # 5*cnt >= 4*size is the exact rational form of cnt/size >= 0.8
    expectDV = (5 * np.maximum(0, 44 - k) >= 4 * (L - k)).astype(np.uint8)
    assert np.array_equal(hm.D, expectDV) and np.array_equal(hm.V, expectDV)


# ---- injected score tensors (closed forms for counts, match and extension) ----------------------------
def _band_tensor(L, w):
    i, j = np.indices((L, L))
    return ((i - j >= 0) & (i - j < w)).astype(np.float32)


def test_injected_band():
    L, w, mu = 256, 32, 0.8
    hm = orc.head_mask_from_probs(_band_tensor(L, w), S=1000, tau=0.3, mu=mu)
    assert np.array_equal(np.flatnonzero(hm.D), np.arange(w))
    # column c has min(L - c, w) cells on it out of L - c: matched iff min(L-c, w) >= mu (L-c),
    # i.e. the last floor(w / mu) = 40 columns (the boundary column has exactly 32 of 40 cells)
    assert np.array_equal(np.flatnonzero(hm.V), np.arange(L - 40, L))
    assert hm.cntV[L - 40] == 32 and hm.cntV[L - 41] == 32
    # extended rows: diagonals continue, the edge columns become verticals for every later row
    rows = [L, L + 5, 700, 999]
    E = hm.rows(rows)
    for a, i in enumerate(rows):
        expect = np.zeros(1000, np.uint8)
        expect[i - w + 1: i + 1] = 1
        expect[L - 40: L] = 1
        assert np.array_equal(E[a], expect), i


def test_injected_sink():
    L = 64
    P = np.zeros((L, L), np.float32)
    P[:, 0] = 1.0
    hm = orc.head_mask_from_probs(P, S=200, tau=0.3, mu=0.8)
    assert np.flatnonzero(hm.V).tolist() == [0]
    # every diagonal has exactly one cell on column 0; only the one-cell diagonal r = L-1 reaches mu
    assert np.flatnonzero(hm.D).tolist() == [L - 1]
    E = hm.rows([L, 150])
    assert np.flatnonzero(E[0]).tolist() == [0, 1]
    assert np.flatnonzero(E[1]).tolist() == [0, 150 - (L - 1)]
    # min_support > 1 (opt-in, not the paper's rule) drops the one-cell diagonal
    hm2 = orc.head_mask_from_probs(P, S=200, tau=0.3, mu=0.8, min_support=2)
    assert np.flatnonzero(hm2.D).tolist() == []


@pytest.mark.parametrize("mu", [0.8, 0.7, 1.0, 0.5])
def test_match_tie_break(mu):
    """A diagonal with ceil(mu*size) cells matches (ties included), one cell fewer does not."""
    L, r = 100, 20
    size = L - r
    need = math.ceil(mu * size - 1e-9)
    for n, expect in ((need, 1), (need - 1, 0)):
        P = np.zeros((L, L), np.float32)
        for t in range(n):
            P[r + t, t] = 1.0
        hm = orc.head_mask_from_probs(P, S=L, tau=0.3, mu=mu)
        assert hm.cntD[r] == n
        assert hm.D[r] == expect


def test_mu_extremes():
    rng = np.random.default_rng(5)
    L = 48
    P = np.tril(rng.random((L, L))).astype(np.float32)
    hm = orc.head_mask_from_probs(P, S=2 * L, tau=0.3, mu=0.0)
    assert hm.D.all() and hm.V.all()
    E = hm.rows(list(range(L, 2 * L)))
    i = np.arange(L, 2 * L)[:, None]
    j = np.arange(2 * L)[None, :]
    assert np.array_equal(E, (j <= i).astype(np.uint8))      # S <= 2L: later rows become fully causal
    hm = orc.head_mask_from_probs(P, S=2 * L, tau=0.3, mu=1.0001)
    assert not hm.D.any() and not hm.V.any()
    assert not hm.rows(list(range(L, 2 * L))).any()


# ---- brute force from the literal pattern matrices ----------------------------------------------------
def _brute_extended(M, S, mu):
    """Sec. 4.2.4 / 4.3 taken literally: every pattern is an L x L 0/1 matrix, its score the ratio of two
    double sums; matched patterns are re-drawn at size S x S and OR-ed below the window."""
    L = M.shape[0]
    out = np.zeros((S, S), np.uint8)
    out[:L, :L] = M
    ii, jj = np.indices((L, L))
    II, JJ = np.indices((S, S))
    ext = np.zeros((S, S), bool)
    for r in range(L):
        Pk = (jj == ii - r)
        # gamma = sum(M * P_k) / sum(P_k) >= mu, in exact integers (mu is a multiple of 0.1 here)
        if (M * Pk).sum() * 10 >= round(mu * 10) * Pk.sum():
            ext |= (JJ == II - r)
    for c in range(L):
        Pk = (jj == c) & (ii >= c)
        if (M * Pk).sum() * 10 >= round(mu * 10) * Pk.sum():
            ext |= (JJ == c) & (II >= c)
    out[L:, :] = ext[L:, :]
    return out


@pytest.mark.parametrize("seed,mu", [(0, 0.8), (1, 0.5), (2, 0.9)])
def test_brute_force_pattern_matrices(seed, mu):
    rng = np.random.default_rng(seed)
    L, S, d = 24, 70, 8
    # structured + random map so that some patterns match and some do not
    Q = rng.standard_normal((L, d)).astype(np.float32)
    K = rng.standard_normal((L, d)).astype(np.float32)
    K[0] += 3 * Q.mean(0)
    P = orc.window_probs(Q, K, L, 1.0)
    P = 0.5 * P + 0.5 * (_band_tensor(L, 3).astype(np.float64) / 3)
    hm = orc.head_mask_from_probs(P, S=S, tau=0.3, mu=mu)
    assert hm.D.any() or hm.V.any()
    full = hm.rows(list(range(S)))
    assert np.array_equal(full, _brute_extended(hm.M, S, mu))


def test_case1_short_sequence_uses_true_mask():
    rng = np.random.default_rng(6)
    L = 32
    P = np.tril(rng.random((L, L))).astype(np.float32)
    hm = orc.head_mask_from_probs(P, S=L, tau=0.3, mu=0.8)
    assert np.array_equal(hm.rows(list(range(L))), hm.M)


# ---- extension invariants -----------------------------------------------------------------------------
def test_extension_invariants():
    rng = np.random.default_rng(7)
    L, S = 40, 200
    P = (np.tril(rng.random((L, L))) * 0.1).astype(np.float32)
    P += _band_tensor(L, 5)
    P[:, 3] = 1.0
    P = np.tril(P).astype(np.float32)
    hm = orc.head_mask_from_probs(P, S=S, tau=0.3, mu=0.8)
    assert hm.D.any() and hm.V.any()
    E = hm.rows(list(range(S)))
    i, j = np.indices((S, S))
    assert not E[j > i].any()                                   # nothing above the diagonal
    assert np.array_equal(E[:L, :L], hm.M)                      # window block untouched
    # Toeplitz beyond the window columns; constant columns inside them
    assert np.array_equal(E[L:-1, L:-1], E[L + 1:, L + 1:])
    for a in range(L, S - 1):
        n = min(L, a - L + 1)
        assert np.array_equal(E[a, :n], E[a + 1, :n])
    # keys in [L, i-L] can never be active for a row i >= L
    for a in range(2 * L, S):
        assert not E[a, L: a - L + 1].any()
    # from row 2L-1 on, verticals and diagonals cannot overlap
    for a in range(2 * L - 1, S):
        assert E[a].sum() == hm.D.sum() + hm.V.sum()


def test_monotone_in_tau_and_mu():
    rng = np.random.default_rng(8)
    L, S, d = 64, 160, 8
    Q = rng.standard_normal((L, d)).astype(np.float32)
    K = rng.standard_normal((L, d)).astype(np.float32)
    P = orc.window_probs(Q, K, L, 1.0)
    prev = None
    for tau in (0.05, 0.1, 0.3, 0.6):
        hm = orc.head_mask_from_probs(P, S=S, tau=tau, mu=0.8)
        if prev is not None:
            assert np.all(hm.M <= prev.M)
        prev = hm
    prev = None
    for mu in (0.2, 0.5, 0.8, 1.0):
        hm = orc.head_mask_from_probs(P, S=S, tau=0.1, mu=mu)
        if prev is not None:
            assert np.all(hm.D <= prev.D) and np.all(hm.V <= prev.V)
            assert np.all(hm.rows(list(range(S))) <= prev.rows(list(range(S))))
        prev = hm


def test_one_cell_patterns():
    rng = np.random.default_rng(9)
    L = 32
    for _ in range(4):
        P = np.tril(rng.random((L, L)) * 0.06).astype(np.float32)
        hm = orc.head_mask_from_probs(P, S=L, tau=0.3, mu=0.8)
        assert hm.V[L - 1] == hm.M[L - 1, L - 1]
        assert hm.D[L - 1] == hm.M[L - 1, 0]


# ---------------------------------------------------------------------------------------------
# Multi-sample averaged map (Sec. 4.2.2)
# ---------------------------------------------------------------------------------------------
def test_capture_average_hand_example():
    # three inputs of lengths 1, 2, 3 and a window of 3: every cell is the mean over the inputs that contain it
    P1 = np.array([[1.0]])
    P2 = np.array([[1.0, 0.0], [0.25, 0.75]])
    P3 = np.array([[1.0, 0.0, 0.0], [0.5, 0.5, 0.0], [0.2, 0.3, 0.5]])
    Abar, C = orc.capture_average([P1, P2, P3], 3, 1e-10)
    assert C.tolist() == [3, 2, 1]
    want = np.array([[1.0, 0.0, 0.0], [0.375, 0.625, 0.0], [0.2, 0.3, 0.5]])
    assert np.allclose(Abar, want, atol=1e-9)
    assert np.allclose(Abar.sum(axis=1), 1.0, atol=1e-9)          # a mean of distributions is a distribution


def test_capture_average_of_copies_is_the_map_and_window_rows_beyond_all_inputs_are_empty():
    rng = np.random.default_rng(3)
    P = np.tril(rng.random((6, 6))).astype(np.float32)
    P /= P.sum(axis=1, keepdims=True)
    A2, C2 = orc.capture_average([P, P], 8, 1e-8, dtype=np.float32)      # 2 P / 2 is exact in binary
    assert np.array_equal(A2[:6, :6], P) and C2.tolist() == [2] * 6 + [0, 0]
    assert not A2[6:].any() and not A2[:, 6:].any()                        # 0 / (0 + eps) = 0
    # masks of the averaged map of identical inputs = masks of the single input
    m1 = orc.head_mask_from_probs(P, 6, 0.3, 0.8)
    m2 = orc.head_mask_from_probs(np.ascontiguousarray(A2[:6, :6]), 6, 0.3, 0.8)
    assert np.array_equal(m1.M, m2.M) and np.array_equal(m1.D, m2.D) and np.array_equal(m1.V, m2.V)


def test_capture_average_float32_tracks_float64():
    rng = np.random.default_rng(4)
    samples = []
    for L in (5, 9, 9, 7, 3):
        P = np.tril(rng.random((L, L)))
        samples.append((P / P.sum(axis=1, keepdims=True)).astype(np.float32))
    a32, c32 = orc.capture_average(samples, 9, 1e-8, dtype=np.float32)
    a64, c64 = orc.capture_average(samples, 9, 1e-8, dtype=np.float64)
    assert np.array_equal(c32, c64) and c64.tolist() == [5, 5, 5, 4, 4, 3, 3, 2, 2]
    assert np.abs(a32 - a64).max() < 1e-6


# ---------------------------------------------------------------------------------------------
# Other amplifications (Appendix B): each is increasing, so its mask is a threshold on the map at the
# inverse function's value; the inverses below are written out independently of the oracle's forward formulas
# ---------------------------------------------------------------------------------------------
def _inverse_threshold(method, tau, lam, eps):
    if method == "log":
        return eps * math.exp(tau)
    if method == "sqrt":
        return (tau + math.sqrt(eps)) ** 2
    if method == "arcsinh":
        return math.sinh(tau + math.asinh(eps))
    if method in ("average", "sum"):
        return tau + eps
    if method == "boxcox":
        return eps * math.exp(tau) if lam == 0 else (lam * tau + eps ** lam) ** (1.0 / lam)
    if method == "yeo_johnson":
        return (eps + 1.0) * math.exp(tau) - 1.0 if lam == 0 else (lam * tau + (eps + 1.0) ** lam) ** (1.0 / lam) - 1.0
    raise ValueError(method)


@pytest.mark.parametrize("method,lam,tau", [
    ("log", 0.0, 12.0), ("sqrt", 0.0, 0.15), ("arcsinh", 0.0, 0.02), ("average", 0.0, 0.03),
    ("boxcox", 0.5, 0.3), ("boxcox", 0.25, 1.0), ("boxcox", 0.0, 12.0), ("boxcox", 1.0, 0.03),
    ("yeo_johnson", 0.5, 0.02), ("yeo_johnson", 0.0, 0.02), ("yeo_johnson", 2.0, 0.05), ("sum", 0.0, 0.03),
])
def test_transform_mask_is_threshold_at_inverse(method, lam, tau):
    eps = 1e-8
    rng = np.random.default_rng(11)
    L = 96
    P = np.tril(rng.random((L, L)) ** 6)
    P /= P.sum(axis=1, keepdims=True)
    M = orc.true_mask_transform(P, tau, method, lam, eps)
    x = _inverse_threshold(method, tau, lam, eps)
    near = np.abs(P - x) <= 1e-9 * max(x, 1e-30)                   # cells within rounding of the threshold
    want = np.tril(P >= x)
    assert np.array_equal(M.astype(bool) | near, want | near)
    assert 0 < M.sum() < L * (L + 1) // 2                            # the case separates something
    assert not np.triu(M, 1).any()


def test_transform_boxcox_half_equals_the_default_path_and_sqrt_is_its_half():
    rng = np.random.default_rng(12)
    P = np.tril(rng.random((64, 64)) ** 4)
    P /= P.sum(axis=1, keepdims=True)
    A = orc.amplify_transform(P, "boxcox", 0.5, 1e-8)
    assert np.allclose(A, orc.amplify_f64(P, 0.5, 1e-8), atol=1e-12)
    assert np.allclose(A, 2.0 * orc.amplify_transform(P, "sqrt", 0.0, 1e-8), atol=1e-12)   # 2 (sqrt X - sqrt eps)
    assert np.array_equal(orc.true_mask_transform(P, 0.3, "boxcox", 0.5, 1e-8), orc.true_mask_f64(P, 0.3, 0.5, 1e-8))
    # every amplification is zero at its minimum and increasing in the map value
    for m, lam in (("log", 0), ("arcsinh", 0), ("average", 0), ("yeo_johnson", 0.5), ("boxcox", 0.1)):
        T = orc.amplify_transform(P, m, lam, 1e-8)
        assert T.min() == 0.0
        order = np.argsort(P, axis=None)
        assert np.all(np.diff(T.reshape(-1)[order]) >= -1e-15)


def test_raw_sum_of_samples_is_the_average_with_the_threshold_scaled_by_the_count():
    """Appendix B, method 1 (raw sum) against method 2 (average): for n samples that all cover the window the sum is
    n times the average, so thresholding the sum at n * tau keeps the cells the average keeps at tau (eps scaled
    alike); worked out by hand, not through the oracle's own formula."""
    rng = np.random.default_rng(14)
    L, n = 48, 4
    samples = []
    for _ in range(n):
        P = np.tril(rng.random((L, L)) ** 5)
        samples.append(P / P.sum(axis=1, keepdims=True))
    total = np.sum(samples, axis=0)
    M_sum = orc.true_mask_transform(total, n * 0.03, "sum", 0.0, n * 1e-8)
    M_avg = orc.true_mask_transform(total / n, 0.03, "average", 0.0, 1e-8)
    assert np.array_equal(M_sum, M_avg) and 0 < M_sum.sum() < L * (L + 1) // 2


def test_zscore_and_minmax_masks_are_thresholds_on_the_map_statistics():
    """(X - mean) / (std + eps) and (X - min) / (max - min + eps), minus their minima, against the thresholds
    worked out by hand: X >= eps + tau (std + eps) and X >= eps + tau (max - eps + eps)."""
    eps = 1e-8
    rng = np.random.default_rng(21)
    L = 80
    P = np.tril(rng.random((L, L)) ** 5)
    P /= P.sum(axis=1, keepdims=True)
    X = np.maximum(P, eps)                                   # every cell, eps above the diagonal
    mean = X.sum() / X.size
    std = math.sqrt(((X - mean) ** 2).sum() / X.size)        # population deviation, written out
    for method, tau, thr in (("zscore", 1.5, eps + 1.5 * (std + eps)), ("minmax", 0.2, eps + 0.2 * (X.max() - eps + eps))):
        M = orc.true_mask_transform(P, tau, method, 0.0, eps)
        near = np.abs(X - thr) <= 1e-9 * thr
        assert np.array_equal(M.astype(bool) | near, np.tril(X >= thr) | near)
        assert 0 < M.sum() < L * (L + 1) // 2
    A = orc.amplify_transform(P, "minmax", 0.0, eps)
    assert A.min() == 0.0 and 0.999 < A.max() < 1.0          # (max - min) / (max - min + eps)
    Z = orc.amplify_transform(P, "zscore", 0.0, eps)
    assert Z.min() == 0.0 and abs((Z - Z.mean()).std() - std / (std + eps)) < 1e-9
