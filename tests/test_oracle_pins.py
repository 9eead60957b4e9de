"""Pins for the CPU oracle: everything here checks oracle/ against what the
paper prints or what mathematics fixes, never against the CUDA path."""
import math
import os

import numpy as np
import pytest

from oracle import turboquant_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def paper_values():
    vals = {}
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.split("#", 1)[0].split()
            if line:
                vals[line[0]] = [float(v) for v in line[1:]]
    return vals


PAPER = paper_values()


# ---- independent numerics used only by the tests --------------------------
def gauss_legendre(fn, a, b, order=96, panels=8):
    x, w = np.polynomial.legendre.leggauss(order)
    edges = np.linspace(a, b, panels + 1)
    tot = 0.0
    for lo, hi in zip(edges[:-1], edges[1:]):
        tot += 0.5 * (hi - lo) * np.sum(w * fn(0.5 * (hi - lo) * x + 0.5 * (hi + lo)))
    return tot


def density(x, d):
    """Lemma 1's density typed again from its formula (not the oracle's function)."""
    k = math.exp(math.lgamma(d / 2) - math.lgamma((d - 1) / 2)) / math.sqrt(math.pi)
    return k * (1 - x * x) ** ((d - 3) / 2)


def support_edges(d):
    """Effective support: beyond ~12 sigma the density is below 1e-30."""
    r = min(1.0, 12.0 / math.sqrt(d))
    return -r, r


def cost_by_quadrature(d, c):
    """Eq. (4) evaluated cell by cell with Gauss-Legendre."""
    lo, hi = support_edges(d)
    t = np.concatenate(([lo], 0.5 * (c[:-1] + c[1:]), [hi]))
    return sum(gauss_legendre(lambda x, ci=ci: (x - ci) ** 2 * density(x, d), t[i], t[i + 1])
               for i, ci in enumerate(c))


def random_unit(n, d, seed):
    g = np.random.default_rng(seed).standard_normal((n, d))
    return g / np.linalg.norm(g, axis=1, keepdims=True)


# ---- Lemma 1 ---------------------------------------------------------------
@pytest.mark.parametrize("d", [3, 4, 8, 64, 200, 1536])
def test_density_integrates_to_one_and_matches_cdf(d):
    lo, hi = support_edges(d)
    tol = 1e-10 if d >= 8 or d == 3 else 1e-6     # sqrt-type end points slow the quadrature for d = 4
    assert abs(gauss_legendre(lambda x: orc.coordinate_density(x, d), lo, hi) - 1.0) < tol
    for x in (-0.5 / math.sqrt(d), 0.3 / math.sqrt(d), min(0.99, 1.7 / math.sqrt(d))):
        cdf = gauss_legendre(lambda t: density(t, d), lo, x)
        assert abs(cdf - orc.coordinate_cdf(x, d)) < tol


def test_density_is_sphere_coordinate_law():
    d = 8
    y = random_unit(400000, d, 11)[:, 0]
    for x in (-0.6, -0.2, 0.1, 0.5):
        assert abs(np.mean(y <= x) - orc.coordinate_cdf(x, d)) < 4 * 0.5 / math.sqrt(y.size)


# ---- codebook (Eq. 4) --------------------------------------------------------
@pytest.mark.parametrize("d", [2, 3, 8, 64, 128, 200, 1536, 3072])
def test_b1_centroid_closed_form(d):
    # E|X| = Gamma(d/2) / (sqrt(pi) Gamma((d+1)/2)), from int_0^1 x (1-x^2)^((d-3)/2) dx = 1/(d-1)
    closed = math.exp(math.lgamma(d / 2) - math.lgamma((d + 1) / 2)) / math.sqrt(math.pi)
    c = orc.codebook(d, 1)
    assert c.shape == (2,)
    assert abs(c[1] - closed) < 1e-12 and abs(c[0] + closed) < 1e-12
    if d >= 64:   # Section 3.1: -> sqrt(2/(pi d)); relative gap ~ 1/(4d)
        limit = PAPER["centroid_b1_sqrt_d"][0] / math.sqrt(d)
        assert abs(c[1] / limit - 1.0) < 1.0 / (2 * d)
        assert abs((c[1] / limit - 1.0) * 4 * d - 1.0) < 0.2


def test_b2_centroids_large_d_match_paper():
    d = 4096
    c = orc.codebook(d, 2) * math.sqrt(d)
    inner, outer = PAPER["centroids_b2_sqrt_d"]
    assert abs(c[2] - inner) < 1e-3 and abs(c[1] + inner) < 1e-3
    assert abs(c[3] - outer) < 5e-3 and abs(c[0] + outer) < 5e-3


def test_b0_is_single_zero_centroid():
    assert np.array_equal(orc.codebook(128, 0), np.zeros(1))


@pytest.mark.parametrize("d,b", [(8, 2), (64, 3), (200, 2), (1536, 3), (1536, 4), (3072, 1)])
def test_centroids_are_conditional_means_and_sorted(d, b):
    c = orc.codebook(d, b)
    assert c.shape == (1 << b,)
    assert np.all(np.diff(c) > 0) and np.all(np.abs(c) <= 1)
    assert np.max(np.abs(c + c[::-1])) < 1e-15
    lo, hi = support_edges(d)
    t = np.concatenate(([lo], 0.5 * (c[:-1] + c[1:]), [hi]))
    for i in range(c.size):
        num = gauss_legendre(lambda x: x * density(x, d), t[i], t[i + 1])
        den = gauss_legendre(lambda x: density(x, d), t[i], t[i + 1])
        assert abs(num / den - c[i]) < 1e-9 / math.sqrt(d)


@pytest.mark.parametrize("d", [128, 1536])
def test_dmse_values_and_bounds(d):
    printed = PAPER["dmse_b1_b4"]
    unit = [0.01, 0.001, 0.01, 0.001]          # one unit of the last printed digit
    for b in (1, 2, 3, 4):
        c = orc.codebook(d, b)
        dmse = d * cost_by_quadrature(d, c)
        assert abs(dmse - printed[b - 1]) <= unit[b - 1], (b, dmse)
        assert PAPER["lower_const"][0] * 4.0 ** -b <= dmse <= PAPER["dmse_upper_const"][0] * 4.0 ** -b
        if b == 1:
            assert abs(dmse - (1 - d * c[1] ** 2)) < 1e-10          # 1 - d c^2 -> 1 - 2/pi
            assert abs(dmse / 4.0 ** -b - PAPER["ratio_to_lower_b1"][0]) < 0.01


def test_codebook_is_a_local_minimum_of_eq4():
    d, b = 64, 3
    c = orc.codebook(d, b)
    base = cost_by_quadrature(d, c)
    rng = np.random.default_rng(0)
    for _ in range(20):
        p = np.sort(c + rng.standard_normal(c.size) * 1e-3 / math.sqrt(d))
        assert cost_by_quadrature(d, p) > base


def test_codebook_matches_sample_kmeans():
    d, b = 8, 2
    y = np.sort(random_unit(2_000_000, d, 5)[:, 0])
    c = np.linspace(-0.9, 0.9, 1 << b)                  # a different start from the oracle's
    for _ in range(200):
        edges = np.searchsorted(y, 0.5 * (c[:-1] + c[1:]))
        c = np.array([seg.mean() for seg in np.split(y, edges)])
    assert np.max(np.abs(c - orc.codebook(d, b))) < 2e-3


def test_index_probabilities_and_entropy():
    for d, b in [(128, 2), (1536, 4)]:
        p = orc.index_probabilities(d, orc.codebook(d, b))
        assert abs(p.sum() - 1) < 1e-12 and np.all(p > 0)
    p = orc.index_probabilities(1536, orc.codebook(1536, 4))
    entropy = -np.sum(p * np.log2(p))
    assert abs(entropy - PAPER["entropy_b4"][0]) < 0.06
    y = orc.rotate(random_unit(2000, 1536, 1), orc.rotation(1536, 9))
    emp = np.bincount(orc.nearest_centroid(y, orc.codebook(1536, 4)).ravel(), minlength=16) / y.size
    assert np.max(np.abs(emp - p)) < 2e-3


# ---- random draws, rotation ---------------------------------------------------
def test_gaussian_matrix_law_and_determinism():
    g = orc.gaussian_matrix(300, 400, 7)
    assert np.array_equal(g, orc.gaussian_matrix(300, 400, 7))
    assert not np.allclose(g, orc.gaussian_matrix(300, 400, 8))
    assert abs(g.mean()) < 4 / math.sqrt(g.size) and abs(g.var() - 1) < 4 * math.sqrt(2 / g.size)
    assert abs(np.mean(g ** 4) - 3) < 0.1
    s = np.sort(g.ravel())
    ecdf = (np.arange(s.size) + 0.5) / s.size
    normal_cdf = 0.5 * (1 + np.vectorize(math.erf)(s / math.sqrt(2)))
    assert np.max(np.abs(ecdf - normal_cdf)) < 1.95 / math.sqrt(s.size)
    # counter layout: entry (r, c) depends on r*cols + c only
    assert orc.gaussian_matrix(2, 400, 7)[1, 3] == g[1, 3]
    assert abs(np.corrcoef(g[:-1].ravel(), g[1:].ravel())[0, 1]) < 0.02


def test_counter_hash_known_values():
    # SplitMix64 finaliser of 0 and 1, computed by hand-written integer arithmetic
    def mix(x):
        m = (1 << 64) - 1
        x ^= x >> 30
        x = (x * 0xBF58476D1CE4E5B9) & m
        x ^= x >> 27
        x = (x * 0x94D049BB133111EB) & m
        return x ^ (x >> 31)
    g = 0x9E3779B97F4A7C15
    m = (1 << 64) - 1
    for seed in (0, 42, 2 ** 63 + 5):
        for ctr in (0, 1, 123456789):
            want = mix((mix((seed + g) & m) + ctr * g) & m)
            assert int(orc.counter_u64(seed, np.array([ctr], dtype=np.uint64))[0]) == want


@pytest.mark.parametrize("d", [5, 64, 200, 512])
def test_rotation_is_orthogonal(d):
    P = orc.rotation(d, 42)
    assert np.max(np.abs(P @ P.T - np.eye(d))) < 1e-12
    assert np.max(np.abs(P.T @ P - np.eye(d))) < 1e-12
    # QR of the same Gaussian matrix: Pi^T G must be upper triangular with positive diagonal
    R = P.T @ orc.gaussian_matrix(d, d, 42)
    assert np.max(np.abs(np.tril(R, -1))) < 1e-10 and np.all(np.diag(R) > 0)


def test_rotated_coordinates_follow_lemma1():
    d = 512
    x = np.zeros((1, d))
    x[0, 3] = 1.0                                         # a worst-case (axis-aligned) input
    y = np.sort(orc.rotate(x, orc.rotation(d, 3))[0])
    ecdf = (np.arange(d) + 0.5) / d
    assert np.max(np.abs(ecdf - orc.coordinate_cdf(y, d))) < 1.63 / math.sqrt(d)
    assert abs(np.sum(y * y) - 1) < 1e-12


# ---- packing --------------------------------------------------------------------
def test_pack_bits_worked_examples():
    assert orc.pack_bits(np.array([[1, 2, 3, 0]]), 2, 4).tolist() == [[0x39, 0, 0, 0]]
    assert orc.pack_bits(np.array([[5, 1, 7]]), 3, 4).tolist() == [[0xCD, 0x01, 0, 0]]
    assert orc.pack_bits(np.array([[1, 0, 0, 0, 0, 0, 0, 1, 1]]), 1, 2).tolist() == [[0x81, 0x01]]
    assert orc.pack_bits(np.array([[15, 1]]), 4, 1).tolist() == [[0x1F]]


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_pack_unpack_round_trip(bits):
    rng = np.random.default_rng(bits)
    v = rng.integers(0, 1 << bits, size=(37, 203)).astype(np.uint8)
    rb = -(-203 * bits // 128) * 16
    p = orc.pack_bits(v, bits, rb)
    assert p.shape == (37, rb)
    assert np.array_equal(orc.unpack_bits(p, bits, 203), v)
    used = 203 * bits
    assert not p[:, (used + 7) // 8:].any()


# ---- Algorithm 1 -------------------------------------------------------------------
def test_quant_mse_matches_python_loops():
    d, b, n = 5, 2, 40
    P = orc.rotation(d, 1)
    c = orc.codebook(d, b)
    X = np.random.default_rng(3).standard_normal((n, d)) * 3.0
    idx, nu = orc.quant_mse(X, P, c)
    for i in range(n):
        norm = math.sqrt(sum(float(v) ** 2 for v in X[i]))
        assert abs(norm - nu[i]) < 1e-12
        for j in range(d):
            yj = sum(float(P[j, k]) * float(X[i, k]) / norm for k in range(d))
            best = min(range(1 << b), key=lambda k: (abs(yj - float(c[k])), k))
            assert best == idx[i, j]


def test_nearest_centroid_tie_and_zero_vector():
    c = np.array([-0.75, -0.25, 0.25, 0.75])             # exactly representable, so ties are exact
    y = np.array([[0.0, 0.5, -0.5, 1.0, -1.0]])
    assert orc.nearest_centroid(y, c).tolist() == [[1, 2, 0, 3, 0]]
    P = orc.rotation(8, 0)
    idx, nu = orc.quant_mse(np.zeros((1, 8)), P, orc.codebook(8, 2))
    assert nu[0] == 0 and idx.tolist() == [[1] * 8]
    assert np.array_equal(orc.dequant_mse(idx, nu, P, orc.codebook(8, 2)), np.zeros((1, 8)))


@pytest.mark.parametrize("b", [1, 2, 3, 4])
def test_dequant_mse_distortion_identity_and_level(b):
    d, n = 256, 4000
    P = orc.rotation(d, 10 + b)
    c = orc.codebook(d, b)
    X = random_unit(n, d, b) * np.random.default_rng(b).uniform(0.5, 4.0, size=(n, 1))
    idx, nu = orc.quant_mse(X, P, c)
    Xh = orc.dequant_mse(idx, nu, P, c)
    # ||x - x~|| = ||Pi x - y~|| because Pi is a rotation (proof of Theorem 1)
    Y = orc.rotate(X / nu[:, None], P)
    lhs = np.linalg.norm(X - Xh, axis=1)
    rhs = np.linalg.norm(Y - c[idx], axis=1) * nu
    assert np.max(np.abs(lhs - rhs)) < 1e-12
    dmse = np.mean((lhs / nu) ** 2)
    assert abs(dmse / (d * cost_by_quadrature(d, c)) - 1) < 0.03
    assert 4.0 ** -b <= dmse <= PAPER["dmse_upper_const"][0] * 4.0 ** -b
    if b == 1:  # Section 3.2: Q^-1(z) = c Pi^T z with z = sign(Pi x)
        assert np.allclose(Xh, c[1] * nu[:, None] * (np.sign(Y) @ P), atol=1e-13)


def test_dmse_is_data_oblivious():
    """Same distortion on a strongly anisotropic, offset law (Section 1.1: worst-case inputs)."""
    d, b, n = 256, 2, 4000
    rng = np.random.default_rng(8)
    W = rng.standard_normal((n, d)) * np.arange(1, d + 1) ** -0.5
    W /= np.linalg.norm(W, axis=1, keepdims=True)
    mu = rng.standard_normal(d)
    W += 0.3 * mu / np.linalg.norm(mu)
    W /= np.linalg.norm(W, axis=1, keepdims=True)
    P, c = orc.rotation(d, 77), orc.codebook(d, b)
    idx, nu = orc.quant_mse(W, P, c)
    dmse = np.mean(np.sum((W - orc.dequant_mse(idx, nu, P, c)) ** 2, axis=1))
    assert abs(dmse / (d * cost_by_quadrature(d, c)) - 1) < 0.05


def test_mse_estimator_bias_at_one_bit():
    d, n = 256, 20000
    P, c = orc.rotation(d, 5), orc.codebook(d, 1)
    X = random_unit(n, d, 21)
    idx, nu = orc.quant_mse(X, P, c)
    est = np.sum(X * orc.dequant_mse(idx, nu, P, c), axis=1)      # <x, x~>, truth = 1
    assert abs(est.mean() / PAPER["mse_bias_b1"][0] - 1) < 0.01
    # bias fades with more bits (Section 4.1)
    c4 = orc.codebook(d, 4)
    idx4, _ = orc.quant_mse(X[:2000], P, c4)
    assert abs(np.sum(X[:2000] * orc.dequant_mse(idx4, nu[:2000], P, c4), axis=1).mean() - 1) < 0.02


# ---- Definition 1 / Algorithm 2 -------------------------------------------------------
def _prod_trials(d, b, trials, rho):
    """Estimator error over independent (Pi, S) draws for one fixed pair (x, y)."""
    x = np.zeros((1, d)); x[0, 0] = 1.0
    y = np.zeros((1, d)); y[0, 0] = rho; y[0, 1] = math.sqrt(1 - rho * rho)
    c = orc.codebook(d, b - 1)
    err, gam = np.empty(trials), np.empty(trials)
    for t in range(trials):
        P, S = orc.rotation(d, 1000 + 2 * t), orc.projection(d, 1001 + 2 * t)
        idx, z, gamma, nu = orc.quant_prod(x, P, S, c)
        xh = orc.dequant_prod(idx, z, gamma, nu, P, S, c)
        err[t] = orc.score(y, xh)[0, 0] - rho
        gam[t] = gamma[0]
    return err, gam


@pytest.mark.parametrize("b,rho", [(1, 0.0), (2, 0.6), (3, 0.3)])
def test_prod_estimator_unbiased_and_within_bounds(b, rho):
    d, trials = 16, 6000
    err, gam = _prod_trials(d, b, trials, rho)
    assert abs(err.mean()) < 4 * err.std() / math.sqrt(trials)
    dprod = np.mean(err ** 2)
    assert dprod <= PAPER["dprod_upper_const"][0] / d / 4.0 ** b
    # conditional variance bound of the proof of Theorem 2: <= pi/(2d) ||y||^2 E||r||^2
    assert dprod <= PAPER["qjl_var_const"][0] / d * np.mean(gam ** 2) * 1.08
    if b == 1:
        assert np.allclose(gam, 1.0)                       # zero-bit MSE stage: r = x
        assert abs(dprod * d / PAPER["dprod_times_d_b1_b4"][0] - 1) < 0.08


def test_wrong_qjl_scale_would_break_unbiasedness():
    """The unbiasedness pin is sensitive: dropping sqrt(pi/2) biases the estimate by ~ -20 % of <y, r>."""
    d, trials, rho = 16, 3000, 0.9
    x = np.zeros((1, d)); x[0, 0] = 1.0
    y = np.zeros((1, d)); y[0, 0] = rho; y[0, 1] = math.sqrt(1 - rho * rho)
    err = np.empty(trials)
    for t in range(trials):
        S = orc.projection(d, 5000 + t)
        z, _ = orc.qjl_quant(x, S)
        err[t] = (y @ (z @ S).T)[0, 0] / d - rho           # planted mistake: no sqrt(pi/2)
    assert abs(err.mean()) > 6 * err.std() / math.sqrt(trials)


@pytest.mark.parametrize("b", [2, 3, 4, 5])
def test_prod_residual_energy_and_distortion_large_d(b):
    d, n = 256, 3000
    P, S, c = orc.rotation(d, 31), orc.projection(d, 32), orc.codebook(d, b - 1)
    X = random_unit(n, d, 40 + b)
    Yq = random_unit(n, d, 50 + b)
    idx, z, gamma, nu = orc.quant_prod(X, P, S, c)
    assert np.allclose(nu, 1.0)
    dmse_prev = d * cost_by_quadrature(d, c)
    assert abs(np.mean(gamma ** 2) / dmse_prev - 1) < 0.03      # E||r||^2 = D_mse(b-1)
    Xh = orc.dequant_prod(idx, z, gamma, nu, P, S, c)
    err = np.sum(Yq * Xh, axis=1) - np.sum(Yq * X, axis=1)
    dprod = np.mean(err ** 2)
    assert 4.0 ** -b / d <= dprod <= PAPER["dprod_upper_const"][0] / d / 4.0 ** b
    assert abs(dprod / (math.pi / 2 / d * dmse_prev) - 1) < 0.12  # chain in the proof of Theorem 2
    if b <= 4:
        assert abs(dprod * d / PAPER["dprod_times_d_b1_b4"][b - 1] - 1) < 0.25
    assert abs(err.mean()) < 4 * err.std() / math.sqrt(n)


def test_qjl_lemma_single_vector():
    d, trials = 32, 4000
    x = random_unit(1, d, 1); y = random_unit(1, d, 2) * 2.0
    est = np.empty(trials)
    for t in range(trials):
        S = orc.projection(d, 9000 + t)
        z, p = orc.qjl_quant(x, S)
        assert np.array_equal(z[0] > 0, (S @ x[0]) >= 0)
        est[t] = (y @ orc.qjl_dequant(z, S).T)[0, 0]
    truth = float((y @ x.T)[0, 0])
    assert abs(est.mean() - truth) < 4 * est.std() / math.sqrt(trials)
    assert est.var() <= PAPER["qjl_var_const"][0] / d * 4.0 * 1.05


def test_qjl_sign_of_zero_is_plus_one():
    z, _ = orc.qjl_quant(np.zeros((1, 4)), orc.projection(4, 0))
    assert z.tolist() == [[1, 1, 1, 1]]


def test_transposed_rotation_in_dequant_would_be_caught():
    d, b = 64, 3
    P, c = orc.rotation(d, 2), orc.codebook(d, b)
    X = random_unit(200, d, 3)
    idx, nu = orc.quant_mse(X, P, c)
    wrong = c[idx] @ P.T                                      # planted mistake: Pi instead of Pi^T
    assert np.mean(np.sum((X - wrong) ** 2, axis=1)) > 1.0    # versus ~0.03 for the right one


# ---- scan side ----------------------------------------------------------------------------
def test_topk_against_sorted():
    rng = np.random.default_rng(0)
    s = rng.integers(0, 20, size=(5, 300)).astype(np.float64)   # many ties
    vals, ids = orc.topk(s, 17)
    for r in range(5):
        want = sorted(range(300), key=lambda i: (-s[r, i], i))[:17]
        assert ids[r].tolist() == want and vals[r].tolist() == [s[r, i] for i in want]


def test_attend_is_softmax_average():
    rng = np.random.default_rng(1)
    s, v = rng.standard_normal((3, 50)), rng.standard_normal((50, 7))
    out = orc.attend(s, v, 0.25)
    for r in range(3):
        w = [math.exp(0.25 * s[r, t]) for t in range(50)]
        for k in range(7):
            assert abs(sum(w[t] * v[t, k] for t in range(50)) / sum(w) - out[r, k]) < 1e-12


def test_outlier_channel_rule():
    X = np.ones((10, 6)); X[:, 4] = 3; X[:, 1] = 2; X[:, 5] = 2
    assert orc.select_outlier_channels(X, 2).tolist() == [1, 4]
    assert orc.select_outlier_channels(X, 3).tolist() == [1, 4, 5]


# ------------------------------------------------------------------ entropy coding of the indices
def test_huffman_on_dyadic_probabilities_has_the_textbook_lengths():
    # p = 2^-len exactly: the optimal code assigns exactly -log2 p bits
    assert orc.huffman_lengths([0.5, 0.25, 0.125, 0.125]).tolist() == [1, 2, 3, 3]
    assert orc.huffman_lengths([0.125, 0.5, 0.125, 0.25]).tolist() == [3, 1, 3, 2]
    assert orc.huffman_lengths([0.25] * 4).tolist() == [2, 2, 2, 2]


def test_canonical_codes_follow_the_published_worked_example():
    # RFC 1951, section 3.2.2: symbols A..H with lengths (3, 3, 3, 3, 3, 2, 4, 4)
    codes = orc.canonical_codes([3, 3, 3, 3, 3, 2, 4, 4])
    assert codes.tolist() == [0b010, 0b011, 0b100, 0b101, 0b110, 0b00, 0b1110, 0b1111]


@pytest.mark.parametrize("d,b", [(1536, 4), (1536, 3), (200, 2), (64, 3)])
def test_huffman_code_of_the_index_distribution(d, b):
    c = orc.codebook(d, b)
    p = orc.index_probabilities(d, c)
    lengths = orc.huffman_lengths(p)
    assert sum(2.0 ** -int(l) for l in lengths) == 1.0                      # Kraft equality: a complete prefix code
    entropy = float(-(p * np.log2(p)).sum())
    avg = float((p * lengths).sum())
    assert entropy <= avg < entropy + 1.0                                     # optimal prefix code
    order = np.argsort(-p, kind="stable")
    assert np.all(np.diff(lengths[order].astype(int)) >= 0)                   # a likelier index never has the longer code
    # no other length assignment satisfying Kraft does better (all assignments with lengths <= 8 at b <= 2)
    if b <= 2:
        import itertools
        best = min(float((p * np.array(ls)).sum()) for ls in itertools.product(range(1, 6), repeat=1 << b)
                   if sum(2.0 ** -l for l in ls) <= 1.0)
        assert abs(best - avg) < 1e-12
    if (d, b) == (1536, 4):
        # Section 3.1: the entropy is about 3.8 bits at b = 4 and coding saves about 5 % of the bit width
        assert abs(entropy - 3.8) < 0.05 and 0.03 < (4.0 - avg) / 4.0 < 0.07


def test_entropy_row_stream_worked_example_and_round_trip():
    lengths = np.array([2, 1, 3, 3], dtype=np.uint8)
    codes = orc.canonical_codes(lengths)
    assert codes.tolist() == [0b10, 0b0, 0b110, 0b111]
    # symbols 1, 0, 3, 2, 1 -> bits 0 | 1 0 | 1 1 1 | 1 1 0 | 0, stream position p = bit (p & 7) of byte (p >> 3):
    # byte 0 holds 0,1,0,1,1,1,1,1 from its least significant bit = 2 + 8 + 16 + 32 + 64 + 128 = 250; byte 1 holds 0,0
    stream, nbits = orc.entropy_encode_row([1, 0, 3, 2, 1], lengths, codes)
    assert nbits == 10
    assert stream.tolist() == [250, 0]
    assert orc.entropy_decode_row(stream, 5, lengths, codes).tolist() == [1, 0, 3, 2, 1]
    rng = np.random.default_rng(0)
    c = orc.codebook(256, 4)
    p = orc.index_probabilities(256, c)
    ln = orc.huffman_lengths(p)
    cd = orc.canonical_codes(ln)
    sym = rng.choice(16, size=500, p=p / p.sum())
    st, nb = orc.entropy_encode_row(sym, ln, cd)
    assert nb == int(ln[sym].sum())
    assert np.array_equal(orc.entropy_decode_row(st, 500, ln, cd), sym)
