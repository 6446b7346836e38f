"""Pins of the CPU oracle's level fit and of its QODA loop (no CUDA involved).

The paper gives the fit's objective but no solver, so the solver is pinned only through
properties of that objective; the QODA update is pinned through the identities of the
paper's appendix and through its behaviour on bilinear games.
"""
import math

import numpy as np
import pytest

SEED = 0x5EED0DA


def _hist_of(orc, u):
    """Histogram of given normalised magnitudes (norm 1 under the max norm)."""
    v = np.asarray(u, np.float32)
    v = np.concatenate([v, np.float32([1.0])])              # makes the max norm exactly 1
    h = orc.histogram_layer(v, 1.0)
    h[385] -= 1
    return h


def _sample_objective(u, levels):
    """(1/d) sum_i (l_{tau+1}-u_i)(u_i-l_tau): Eq. (Var) per unit squared norm, from the samples."""
    lv = np.asarray(levels, np.float64)
    tau = np.clip(np.searchsorted(lv, u, side="right") - 1, 0, len(lv) - 2)
    return float(np.mean((lv[tau + 1] - u) * (u - lv[tau])))


def test_uniform_density_gives_uniform_levels(orc):
    """For a uniform density on [0,1] the stationarity condition reads (b-a)^2 = (c-b)^2,
    so the minimiser is the uniform grid j/(n-1)."""
    N = 1 << 21
    u = (np.arange(N) + 0.5) / N
    h = _hist_of(orc, u)
    for n in (4, 8, 16):
        lv = orc.fit_levels(h[None, :], [1.0], N, n)
        assert np.allclose(lv, np.arange(n) / (n - 1), atol=2e-4)


def test_two_piece_density_has_levels_one_quarter_and_three_fifths(orc):
    """A density that is constant on [0, 1/3] and 5/32 times as high on (1/3, 1].  With four levels {0, b1, b2, 1}
    and b1 < 1/3 < b2 the two first-order conditions of the objective,
        int_0^b1 u dF = int_b1^b2 (b2 - u) dF   and   int_b1^b2 (u - b1) dF = int_b2^1 (1 - u) dF,
    read, with x = 1/3 - b1 and r = 5/32:
        b1^2 / 2 = b2 x - ((1/3)^2 - b1^2) / 2 + r (b2 - 1/3)^2 / 2,
        x^2 / 2 + r ((b2 - b1)^2 - x^2) / 2 = r (1 - b2)^2 / 2.
    b1 = 1/4, b2 = 3/5 solve both exactly (worked out by hand: x = 1/12; 1/32 = 1/20 - 7/288 + (5/64)(16/225), and
    (1/144)(27/32) = (5/32)(0.16 - 0.1225)), and a search from many starting points finds no other minimum."""
    s, r = 1.0 / 3.0, 5.0 / 32.0
    mass1 = s / (s + r * (1.0 - s))                              # share of the mass below 1/3
    N = 1 << 22
    q = (np.arange(N) + 0.5) / N                                 # the density's quantiles: an even sample of it
    u = np.where(q < mass1, q / mass1 * s, s + (q - mass1) / (1.0 - mass1) * (1.0 - s))
    lv = orc.fit_levels(_hist_of(orc, u)[None, :], [1.0], N, 4)
    # (1/3 is not an edge of the histogram's bins, whose content is taken as evenly spread: 1e-3 of slack)
    assert abs(lv[1] - 0.25) < 1e-3 and abs(lv[2] - 0.6) < 1e-3, lv


def test_two_piece_density_with_two_minima_ends_in_the_lower_one(orc):
    """A density that is constant on [0, 3/11] and 4/125 times as high on (3/11, 1].  With four levels the objective
    has two local minima.  b1 = 1/5, b2 = 1/2 satisfies both first-order conditions exactly (by hand:
    b1^2/2 = 1/50 = [u/2 - u^2/2] from 1/5 to 3/11 + (2/125)(5/22)^2, and
    (4/55)^2/2 + (2/125)(9/100 - (4/55)^2) = 1/250 = (4/125)(1/2)^2/2); the other, near (0.136, 0.272), is what
    coordinate descent from the quantile start reaches and is 4 % worse.  The global minimum is found here by brute
    force on the closed-form objective of the continuous density, not by the oracle."""
    s, r = 3.0 / 11.0, 4.0 / 125.0

    def cum(x):                                                  # F, first and second moment of the unnormalised density
        lo = np.minimum(x, s)
        hi = np.maximum(x, s)
        return (lo + r * (hi - s), lo ** 2 / 2 + r * (hi ** 2 - s ** 2) / 2, lo ** 3 / 3 + r * (hi ** 3 - s ** 3) / 3)

    def piece(a, c):
        (Fa, Ma, Sa), (Fc, Mc, Sc) = cum(a), cum(c)
        return (a + c) * (Mc - Ma) - (Sc - Sa) - a * c * (Fc - Fa)

    g = np.arange(1, 1000) / 1000.0
    b1, b2 = np.meshgrid(g, g, indexing="ij")
    f = np.where(b1 < b2, piece(0.0, b1) + piece(b1, b2) + piece(b2, 1.0), np.inf)
    i, j = np.unravel_index(np.argmin(f), f.shape)
    assert (g[i], g[j]) == (0.2, 0.5)
    assert f[i, j] < 0.97 * (piece(0.0, 0.1358) + piece(0.1358, 0.2717) + piece(0.2717, 1.0))

    mass1 = s / (s + r * (1.0 - s))
    N = 1 << 22
    q = (np.arange(N) + 0.5) / N
    u = np.where(q < mass1, q / mass1 * s, s + (q - mass1) / (1.0 - mass1) * (1.0 - s))
    lv = orc.fit_levels(_hist_of(orc, u)[None, :], [1.0], N, 4)
    # (3/11 falls inside the histogram bin [17/64, 18/64], whose content is taken as evenly spread: the step is
    # smeared over 1/64, which moves the levels by up to 3e-3; the other minimum is 0.06 and 0.23 away)
    assert abs(lv[1] - 0.2) < 2e-3 and abs(lv[2] - 0.5) < 4e-3, lv


@pytest.mark.parametrize("dist", ["halfnormal", "laplace", "student"])
def test_fit_is_a_minimum_of_the_objective(orc, dist):
    rng = np.random.default_rng(42)
    d = 60000
    x = {"halfnormal": rng.standard_normal(d), "laplace": rng.laplace(size=d),
         "student": rng.standard_t(3, size=d)}[dist].astype(np.float32)
    norm, _ = orc.layer_norm(x, 2)
    u = np.minimum(np.abs(x) * (np.float32(1) / norm), np.float32(1)).astype(np.float64)
    h = orc.histogram_layer(x, norm)
    n = 16
    lv = orc.fit_levels(h[None, :], [norm], d, n)
    assert lv[0] == 0 and lv[-1] == 1 and np.all(np.diff(lv) > 0)
    f_fit = orc.fit_objective(h[None, :], [norm], d, lv)
    # the closed-form objective on the histogram density agrees with the sample sum of Eq. (Var)
    assert abs(f_fit - _sample_objective(u, lv)) < 0.02 * f_fit
    # better than uniform levels and than exponential levels 2^-(n-1-j)
    uni = orc.uniform_levels(4)
    expo = np.concatenate([[0], 2.0 ** -np.arange(n - 2, -1, -1)]).astype(np.float32)
    assert f_fit < orc.fit_objective(h[None, :], [norm], d, uni)
    assert f_fit < orc.fit_objective(h[None, :], [norm], d, expo)
    # local minimum: random feasible perturbations never improve it (beyond rounding)
    for _ in range(200):
        p = lv.astype(np.float64).copy()
        j = rng.integers(1, n - 1)
        p[j] += rng.uniform(-0.3, 0.3) * min(p[j] - p[j - 1], p[j + 1] - p[j])
        assert orc.fit_objective(h[None, :], [norm], d, p.astype(np.float32)) >= f_fit * (1 - 1e-6)
    # an independent optimiser on the sample objective cannot do noticeably better
    from scipy.optimize import minimize

    def obj(z):
        inner = np.sort(1.0 / (1.0 + np.exp(-z)))
        return _sample_objective(u, np.concatenate([[0.0], inner, [1.0]])) * 1e6
    z0 = np.log(lv[1:-1].astype(np.float64) / (1 - lv[1:-1].astype(np.float64)))
    best = minimize(obj, z0 + rng.normal(0, 0.2, n - 2), method="Powell",
                    options=dict(maxiter=1500, xtol=1e-5, ftol=1e-8)).fun / 1e6
    # (the fit sees the samples only through 16 bins per octave, which costs a few per cent
    # in the sparse tail of heavy-tailed data)
    assert _sample_objective(u, lv) <= best * 1.08


def test_stationarity_condition(orc):
    """At the fitted levels int_a^b (u-a) dF = int_b^c (c-u) dF for every interior level,
    evaluated directly on the samples."""
    rng = np.random.default_rng(7)
    d = 400000
    x = rng.laplace(size=d).astype(np.float32)
    norm, _ = orc.layer_norm(x, 2)
    u = np.abs(x.astype(np.float64)) / float(norm)
    h = orc.histogram_layer(x, norm)
    lv = orc.fit_levels(h[None, :], [norm], d, 8).astype(np.float64)
    for j in range(1, 7):
        a, b, c = lv[j - 1], lv[j], lv[j + 1]
        lo, hi = (u >= a) & (u < b), (u >= b) & (u < c)
        if min(lo.sum(), hi.sum()) < 1000:        # too few samples for a meaningful comparison
            continue
        left, right = np.sum((u - a)[lo]), np.sum((c - u)[hi])
        assert abs(left - right) < 0.01 * max(left, right)


def test_layerwise_fit_beats_shared_fit(orc):
    """Remark after Eq. (MQV): per-layer sequences never lose to one shared sequence."""
    rng = np.random.default_rng(3)
    d = 100000
    xa = rng.standard_normal(d).astype(np.float32)
    xb = (rng.standard_t(3, size=d) * 0.01).astype(np.float32)
    na, _ = orc.layer_norm(xa, 2); nb, _ = orc.layer_norm(xb, 2)
    ha = orc.histogram_layer(xa, na); hb = orc.histogram_layer(xb, nb)
    la = orc.fit_levels(ha[None], [na], d, 8); lb = orc.fit_levels(hb[None], [nb], d, 8)
    # shared sequence: fitted on both samples as one type (weights = squared norms)
    shared = orc.fit_levels(np.stack([ha, hb]), [na, nb], d, 8)
    wa, wb = float(na) ** 2, float(nb) ** 2

    def total(l1, l2):
        return wa * orc.fit_objective(ha[None], [na], d, l1) + wb * orc.fit_objective(hb[None], [nb], d, l2)
    assert total(la, lb) <= total(shared, shared) * (1 + 1e-9)


def test_fit_weights_follow_squared_norms(orc):
    rng = np.random.default_rng(5)
    d = 50000
    xa = rng.standard_normal(d).astype(np.float32); xb = rng.laplace(size=d).astype(np.float32)
    na, _ = orc.layer_norm(xa, 2); nb, _ = orc.layer_norm(xb, 2)
    ha = orc.histogram_layer(xa, na); hb = orc.histogram_layer(xb, nb)
    only_a = orc.fit_levels(ha[None], [na], d, 8)
    both = orc.fit_levels(np.stack([ha, hb]), [na, 0.0], d, 8)       # lambda_b = 0
    assert np.array_equal(only_a, both)
    heavy = orc.fit_levels(np.stack([ha, hb]), [na * 1000, nb], d, 8)  # lambda_b = 1e-6
    assert np.allclose(heavy, only_a, rtol=1e-3)
    assert orc.fit_levels(np.stack([ha, hb]), [0.0, 0.0], d, 8) is None


# ---------------------------------------------------------------------------------- QODA
def _bilinear_operator(A, z):
    n = A.shape[0]
    x, y = z[:n].astype(np.float64), z[n:].astype(np.float64)
    return np.concatenate([A @ y, -(A.T @ x)])


def test_optimism_converges_where_dual_averaging_does_not(orc):
    """min_x max_y xy, exact operator, K = 1, no quantization: the extrapolated (optimistic)
    iterates approach the saddle point, plain dual averaging with the same step rule does not."""
    A = np.array([[1.0]])
    X1 = np.array([1.0, 1.0], np.float32)
    Y = np.zeros(2, np.float32); Xh = X1.copy(); X = X1.copy()
    S, eta = 0.0, np.float32(1.0)
    prev = None
    for t in range(3000):
        V = _bilinear_operator(A, Xh).astype(np.float32)
        S, eta = orc.step_size(S, orc.sq_diff(V, prev), 1)
        orc.qoda_update(V, X1, Y, Xh, X, eta)
        prev = V
    assert np.linalg.norm(X) < 0.05 * np.linalg.norm(X1)
    # plain dual averaging: query at X_t itself
    Yd = np.zeros(2); Xd = X1.astype(np.float64); Sd = 0.0; prevd = np.zeros(2)
    for t in range(3000):
        V = _bilinear_operator(A, Xd)
        Sd += np.sum((V - prevd) ** 2); prevd = V
        Yd -= V
        Xd = X1 + Yd / math.sqrt(1 + Sd)
    assert np.linalg.norm(Xd) > 0.5 * np.linalg.norm(X1)


def test_step_size_formula(orc):
    # eta_{t+1} = (1 + sum_s sum_k ||.||^2 / K^2)^(-1/2), accumulated over calls
    S, eta = orc.step_size(0.0, 8.0, 2)
    assert S == 2.0 and eta == np.float32(1 / math.sqrt(3.0))
    S, eta = orc.step_size(S, 4.0, 2)
    assert S == 3.0 and eta == np.float32(0.5)
    a = np.float32([1.0, 2.0, -3.0]); b = np.float32([0.5, 2.0, 1.0])
    assert orc.sq_diff(a, b) == 0.25 + 16.0 and orc.sq_diff(a, None) == 14.0
    # the difference is an fp32 subtraction (the vectors' own precision), its square summed in fp64
    assert orc.sq_diff(np.float32([1.0]), np.float32([2.0 ** -30])) == 1.0
    big = np.float32([3.0] * 4 + [2.0 ** -20]); zero = np.zeros(5, np.float32)
    assert orc.sq_diff(big, zero) == 36.0 + 2.0 ** -40          # fp64 accumulation keeps the small term


def test_qoda_identities_with_quantization(orc):
    """Appendix identity X_t = X_1 - (eta_t / K) sum_{s<t} sum_k V^_{k,s+1/2}, eta non-increasing,
    X_{t+1/2} = X_t - gamma_t * mean_k V^_{k,t-1/2}; and the gap of the ergodic average decreases
    on a noisy bilinear game (Theorem 5.5)."""
    rng = np.random.default_rng(0)
    n = 32; D = 2 * n; K = 4
    A = rng.standard_normal((n, n)) / math.sqrt(n)
    sizes = [16] * 4
    model = orc.OracleModel(sizes, [4] * 4, 2, K, SEED)
    X1 = (rng.standard_normal(D) / math.sqrt(D)).astype(np.float32)
    model.qoda_init(X1)
    total = np.zeros(D); avg = np.zeros(D); etas = []; gaps = {}
    R = float(np.linalg.norm(X1))
    for t in range(1, 1501):
        Xh = model.Xhalf.copy()
        avg += Xh
        F = _bilinear_operator(A, Xh)
        V = (F[None, :] + 0.1 * rng.standard_normal((K, D))).astype(np.float32)
        out = model.quantize(V, t)
        X_before = model.X.copy(); eta_before = model.eta
        gbar = model.qoda_step()
        total += out["decoded"].astype(np.float64).sum(axis=0)
        etas.append(float(model.eta))
        assert np.allclose(model.X, X1 - float(model.eta) / K * total, rtol=0, atol=2e-5)
        assert np.allclose(model.Xhalf, model.X.astype(np.float64) - float(model.eta) * gbar, atol=1e-6)
        if t in (10, 100, 1500):
            zbar = avg / t
            gaps[t] = R * np.linalg.norm(_bilinear_operator(A, zbar))
    assert all(0 < b <= a <= 1 for a, b in zip(etas, etas[1:]))
    assert gaps[1500] < 0.5 * gaps[100] < 0.5 * gaps[10]


# ---------------------------------------------------------------- alternative step sizes
def test_alt_rates_closed_form_and_ordering(orc):
    eta, gamma = orc.alt_rates(3.0, 5.0, 0.25)
    assert eta == np.float32(1.0 / 3.0) and gamma == np.float32(4.0 ** -0.25)
    assert orc.alt_rates(0.0, 0.0, 0.1) == (np.float32(1.0), np.float32(1.0))     # eta_1 = eta_2 = gamma_1 = gamma_2 = 1
    for lam, mu, qh in [(0.5, 0.0, 0.25), (10.0, 3.0, 0.01), (1e6, 1e3, 0.2)]:
        e, g = orc.alt_rates(lam, mu, qh)
        assert 0 < e <= g <= 1                                                     # the extrapolation step is the larger one
    assert orc.sq_norm(np.float32([3.0, -4.0, 2.0 ** -20])) == 25.0 + 2.0 ** -40


def test_alt_schedule_hand_worked_two_steps(orc):
    """One coordinate, K = 1, operator V(x) = x, 8-bit levels so fine that 1 and -1 are levels
    (no rounding noise): X_1 = 1.  Step 1: X_{3/2} = 1, gbar = 1, eta_2 = gamma_2 = 1, X_2 = 0, X_{5/2} = -1,
    lambda_1 = 1, mu_1 = 1.  Step 2: gbar = -1, Y_3 = 0, eta_3 = 3^(-1/2), X_3 = 1, gamma_3 = 2^(-1/4),
    X_{7/2} = 1 + 2^(-1/4); lambda_2 = 2, mu_2 = 2."""
    model = orc.OracleModel([1], [8], 0, 1, SEED)            # max norm: u = 1 is a level, decoded value exact
    model.alt_qhat = 0.25
    model.qoda_init(np.float32([1.0]))
    for want_g, want_x, want_xh, want_lam, want_mu in [
            (1.0, 0.0, -1.0, 1.0, 1.0),
            (-1.0, 1.0, float(np.float32(1.0) + np.float32(2.0 ** -0.25)), 2.0, 2.0)]:
        V = model.Xhalf.copy()[None, :]
        model.quantize(V, model.t)
        g = model.qoda_step()
        assert float(g[0]) == want_g and float(model.X[0]) == want_x
        assert abs(float(model.Xhalf[0]) - want_xh) <= 1e-7
        assert (model.lam, model.mu) == (want_lam, want_mu)
    assert model.eta == np.float32(3.0 ** -0.5) and model.gamma == np.float32(2.0 ** -0.25)


def test_alt_schedule_converges_on_a_noisy_bilinear_game(orc):
    """Bilinear games are not co-coercive; the alternative rates are the ones the paper proves without
    that assumption.  The identity X_{t+1} = X_1 - eta_{t+1} sum_s gbar_s holds and the gap of the ergodic
    average falls."""
    rng = np.random.default_rng(1)
    n = 32; D = 2 * n; K = 4
    A = rng.standard_normal((n, n)) / math.sqrt(n)
    model = orc.OracleModel([16] * 4, [4] * 4, 2, K, SEED)
    model.alt_qhat = 0.25
    X1 = (rng.standard_normal(D) / math.sqrt(D)).astype(np.float32)
    model.qoda_init(X1)
    total = np.zeros(D); avg = np.zeros(D); gaps = {}; R = float(np.linalg.norm(X1))
    for t in range(1, 1501):
        Xh = model.Xhalf.copy(); avg += Xh
        V = (_bilinear_operator(A, Xh)[None, :] + 0.1 * rng.standard_normal((K, D))).astype(np.float32)
        model.quantize(V, t)
        eta_before = float(model.eta)
        g = model.qoda_step()
        total += g.astype(np.float64)
        assert float(model.eta) <= eta_before and float(model.eta) <= float(model.gamma) <= 1.0
        assert np.allclose(model.X, X1 - float(model.eta) * total, rtol=0, atol=2e-5)
        if t in (10, 100, 1500):
            gaps[t] = R * np.linalg.norm(_bilinear_operator(A, avg / t))
    assert gaps[1500] < 0.5 * gaps[100] < 0.5 * gaps[10]


# ------------------------------------------------------------------ code-length accounting
def test_level_probabilities_partition_and_closed_form(orc):
    rng = np.random.default_rng(21)
    # any density, any levels: the hat functions add up to one, so the probabilities add up to the mass
    u = np.abs(rng.standard_normal(40000)) ** 2 * 0.05
    u = u[u < 1.0]
    h = _hist_of(orc, u)
    lv = np.float32([0, 0.01, 0.03, 0.1, 0.2, 0.45, 0.7, 1.0])
    p = orc.level_probabilities(h[None, :], np.float32([1.0]), u.size, lv)
    assert abs(p.sum() - 1.0) < 1e-12 and np.all(p >= 0)
    # uniform density on [2^-4, 1) (whole bins) and levels on bin edges: the integrals are elementary
    hu = np.zeros(512, np.uint32); d = 0
    for i in range(1 + 16 * 20, 385):
        w = int(round((orc.bin_edge(i + 1) - orc.bin_edge(i)) * 2 ** 20)); hu[i] = w; d += w
    lv = np.float32([0.0, 0.0625, 0.25, 0.5, 1.0])
    p = orc.level_probabilities(hu[None, :], np.float32([2.0]), d, lv)
    dens = 1.0 / (1.0 - 0.0625)
    want = [0.0, dens * (0.25 - 0.0625) / 2, dens * ((0.25 - 0.0625) / 2 + 0.25 / 2), dens * (0.25 / 2 + 0.5 / 2), dens * 0.5 / 2]
    assert np.allclose(p, want, rtol=0, atol=1e-12)
    bits, nz = orc.expected_code_length(p, d)
    H = -sum(x * math.log2(x) for x in want[1:4])
    assert nz == d and abs(bits - (32 + d + (H + 1) * d)) < 1e-6
    # the point mass at u = 1 belongs to the last level
    hp = np.zeros(512, np.uint32); hp[385] = 10
    assert orc.level_probabilities(hp[None, :], np.float32([1.0]), 10, lv).tolist() == [0, 0, 0, 0, 1.0]


def test_emitted_indices_follow_the_level_probabilities(orc):
    """Quantizing the vector whose histogram was taken: the frequency of each emitted index approaches p^_j
    (up to the histogram's resolution), and the non-zero count approaches (1 - p^_0) d."""
    rng = np.random.default_rng(22)
    d = 200000
    v = (rng.standard_t(3, d) * 1e-3).astype(np.float32)
    norm, _ = orc.layer_norm(v, 2)
    h = orc.histogram_layer(v, norm)
    lv = orc.fit_levels(h[None, :], np.float32([norm]), d, 16)
    p = orc.level_probabilities(h[None, :], np.float32([norm]), d, lv)
    counts = np.zeros(16)
    R = 20
    for s in range(R):
        idx, _, _ = orc.quantize_layer(v, norm, lv, SEED, 500 + s, 0, 0)
        counts += np.bincount(idx, minlength=16)
    freq = counts / (R * d)
    assert np.all(np.abs(freq - p) < 0.01 * p + 2e-4)
    _, nz = orc.expected_code_length(p, d)
    assert abs((R * d - counts[0]) / R - nz) < 0.01 * nz


# --------------------------------------------------------------- one sequence per type
def test_shared_fit_reduces_to_the_single_layer_fit_and_minimises_the_summed_variance(orc):
    rng = np.random.default_rng(41)
    # one member layer: the same levels as the per-layer fit
    u = np.abs(rng.standard_normal(30000)) * 0.05
    h = _hist_of(orc, u[u < 1])
    a = orc.fit_levels(np.stack([h, h]), np.float32([1.0, 2.0]), u.size, 8)
    b = orc.fit_levels_shared(np.stack([h, h]), np.float32([1.0, 2.0]), [u.size, u.size], 8)
    assert np.allclose(a, b, rtol=1e-6, atol=0)
    # two member layers of different size, norm and shape: the shared sequence minimises
    # sum_s N_s^2 sum_i sigma_Q^2(u_i) against perturbations and beats either layer's own sequence on that sum
    u1 = np.abs(rng.standard_normal(20000)) * 0.02
    u2 = np.abs(rng.laplace(size=5000)) * 0.08; u2 = u2[u2 < 1]
    h1, h2 = _hist_of(orc, u1), _hist_of(orc, u2)
    N = np.float32([3.0, 0.5])
    lv = orc.fit_levels_shared(np.stack([h1, h2]), N, [u1.size, u2.size], 16)

    def total_variance(levels):
        return float(N[0]) ** 2 * u1.size * _sample_objective(u1, levels) + float(N[1]) ** 2 * u2.size * _sample_objective(u2, levels)
    best = total_variance(lv)
    for own in (orc.fit_levels(h1[None], N[:1], u1.size, 16), orc.fit_levels(h2[None], N[1:], u2.size, 16)):
        assert best <= total_variance(own) * 1.001
    for _ in range(30):
        p = lv.astype(np.float64).copy()
        j = int(rng.integers(1, 15))
        p[j] += rng.uniform(-0.3, 0.3) * min(p[j] - p[j - 1], p[j + 1] - p[j])
        assert best <= total_variance(p) * 1.002


def test_fp32_difference_costs_less_than_one_ulp_in_the_statistic(orc):
    """The statistic of Eq. (general_stepsize) takes the difference of two decoded fp32 values in fp32 (one rounding)
    before squaring in fp64.  Against the exact difference (both values converted to fp64 first) every term is off by at
    most a relative 2^-23, and so is the sum; on two successive messages of normal data the sums differ by far less."""
    rng = np.random.default_rng(11)
    d = 200000
    lv = orc.uniform_levels(4)
    decoded = []
    for step, scale in ((1, 1.0), (2, 0.8)):
        v = (rng.standard_normal(d) * scale).astype(np.float32)
        norm, _ = orc.layer_norm(v, 2)
        idx, sg, _ = orc.quantize_layer(v, norm, lv, 7, step, 0, 0)
        decoded.append(orc.decode_layer(idx, sg, norm, lv))
    got = orc.sq_diff(decoded[1], decoded[0])
    exact = float(np.sum((decoded[1].astype(np.float64) - decoded[0].astype(np.float64)) ** 2))
    rel = abs(got - exact) / exact
    assert rel <= 2.0 ** -23
    assert rel <= 1e-7, rel
    print("relative cost of the fp32 difference in the statistic:", rel)
