"""Pins for the float64 oracle: what the paper and the mathematics fix, independent of the
oracle's own formulas (closed forms, invariants, library routines, brute force, a hand-worked
example).  CPU only."""
import itertools
import math
import pathlib

import mpmath
import numpy as np
import pytest
from scipy import integrate, special, stats

from oracle import polarquant_oracle as orc

GOLDEN = pathlib.Path(__file__).parent / "golden"
RNG = np.random.default_rng(20250202)


@pytest.fixture(scope="module")
def cb():
    return orc.fit_codebooks()


# ---------------------------------------------------------------- transform (Definition 1)
@pytest.mark.parametrize("d,L", [(2, 1), (4, 2), (16, 4), (128, 4), (128, 7), (32, 5)])
def test_polar_is_exactly_invertible(d, L):
    y = RNG.standard_normal((500, d))
    y[:, :3] *= 10.0  # outlier channels
    angles, radii = orc.polar(y, L)
    back = orc.inverse_polar(angles, radii)
    assert np.max(np.abs(back - y)) < 1e-12
    # ranges and counts of Definition 1
    assert len(angles) == L and radii.shape[-1] == d >> L
    assert angles[0].min() >= 0.0 and angles[0].max() < 2 * math.pi
    for l in range(1, L):
        assert angles[l].shape[-1] == d >> (l + 1)
        assert angles[l].min() >= 0.0 and angles[l].max() <= math.pi / 2


def test_block_radius_is_block_norm_and_energy_is_kept_per_level():
    d, L = 128, 4
    y = RNG.standard_normal((300, d)) * RNG.uniform(0.1, 30.0, size=(300, 1))
    _, radii = orc.polar(y, L)
    block_norm = np.linalg.norm(y.reshape(300, d // 16, 16), axis=-1)
    assert np.allclose(radii, block_norm, rtol=1e-13, atol=0)
    for l in range(1, 8):
        _, r = orc.polar(y, l)
        assert np.allclose(np.sum(r * r, -1), np.sum(y * y, -1), rtol=1e-13)
    _, r_full = orc.polar(y, 7)  # full log2(d) recursion: a single radius = ||y||
    assert r_full.shape[-1] == 1
    assert np.allclose(r_full[:, 0], np.linalg.norm(y, axis=-1), rtol=1e-13)


def test_d2_is_textbook_polar_coordinates():
    y = RNG.standard_normal((1000, 2))
    angles, radii = orc.polar(y, 1)
    assert np.allclose(radii[:, 0] * np.cos(angles[0][:, 0]), y[:, 0], atol=1e-14)
    assert np.allclose(radii[:, 0] * np.sin(angles[0][:, 0]), y[:, 1], atol=1e-14)
    z = y[:, 0] + 1j * y[:, 1]
    assert np.allclose(np.mod(np.angle(z), 2 * math.pi), angles[0][:, 0], atol=1e-14)
    assert np.allclose(np.abs(z), radii[:, 0], rtol=1e-15)


def test_zero_and_signed_zero_inputs():
    y = np.array([[0.0, 0.0, -0.0, 0.0], [1.0, -0.0, -1.0, -0.0], [-0.0, -0.0, 0.0, -0.0]])
    angles, radii = orc.polar(y, 2)
    assert np.all(np.isfinite(angles[0])) and np.all(angles[0] >= 0) and np.all(angles[0] < 2 * math.pi)
    assert angles[0][0, 0] == 0.0 and radii[0, 0] == 0.0
    assert not np.any(np.signbit(angles[0]))
    assert np.all(orc.inverse_polar(angles, radii)[0] == 0.0)


# ---------------------------------------------------------------- rotation (Section 3.2 footnote)
@pytest.mark.parametrize("d", [16, 128])
def test_rotation_is_orthogonal_and_preserves_geometry(d):
    S = orc.make_rotation(d, seed=7)
    assert np.max(np.abs(S.T @ S - np.eye(d))) < 1e-13
    x, z = RNG.standard_normal((50, d)), RNG.standard_normal((50, d))
    xs, zs = orc.rotate(x, S), orc.rotate(z, S)
    assert np.allclose(np.linalg.norm(xs, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)
    assert np.allclose(np.sum(xs * zs, 1), np.sum(x * z, 1), rtol=1e-10, atol=1e-12)
    assert not np.allclose(orc.make_rotation(d, seed=8), S)  # seed matters
    assert np.array_equal(orc.make_rotation(d, seed=7), S)  # and is reproducible


@pytest.mark.parametrize("d", [2, 16, 128])
def test_structured_preconditioners_are_what_their_definitions_say(d):
    """Section 3.2 / Section 5 ("PolarQuant" without "-R"): the identity, and diag(signs) H / sqrt(d) with the Sylvester
    matrix.  Pinned by the closed form H[i][j] = (-1)^popcount(i & j), by H H^T = d I in exact integers, by the
    fast Walsh-Hadamard butterfly applied to a vector, and by the order-2 matrix written out."""
    rng = np.random.default_rng(d)
    signs = rng.choice([-1.0, 1.0], size=d)
    S = orc.make_structured_rotation(d, "hadamard", signs)
    H = np.rint(S * np.sqrt(d) * signs[:, None]).astype(np.int64)      # undo the scaling and the row signs
    assert np.array_equal(H, [[(-1) ** bin(i & j).count("1") for j in range(d)] for i in range(d)])
    assert np.array_equal(H @ H.T, d * np.eye(d, dtype=np.int64))
    assert np.allclose(S @ S.T, np.eye(d), atol=1e-14) and np.allclose(np.abs(S), d ** -0.5, atol=1e-16)
    x = rng.standard_normal(d)
    y = x * signs                      # y = x . S: sign flips, butterflies, scaling
    h = 1
    while h < d:
        y = y.reshape(-1, 2, h)
        y = np.stack([y[:, 0] + y[:, 1], y[:, 0] - y[:, 1]], axis=1).reshape(-1)
        h *= 2
    assert np.allclose(orc.rotate(x[None], S)[0], y / np.sqrt(d), atol=1e-12)
    if d == 2:
        assert np.allclose(orc.make_structured_rotation(2, "hadamard", [1, -1]), np.array([[1, 1], [-1, 1]]) / np.sqrt(2))
    assert np.array_equal(orc.make_structured_rotation(d, "identity"), np.eye(d))
    with pytest.raises(ValueError):
        orc.make_structured_rotation(12, "hadamard", np.ones(12))


# ---------------------------------------------------------------- densities (Lemma 2)
def _cdf(level, psi):
    """sin^2(psi) ~ Beta(2^(l-2), 2^(l-2)): Lemma 2's density after a change of variable."""
    a = 2.0 ** (level - 2)
    return special.betainc(a, a, np.sin(psi) ** 2)


@pytest.mark.parametrize("level", [2, 3, 4, 5])
def test_density_matches_lemma2_constants_and_beta_cdf(level):
    total, _ = integrate.quad(lambda p: float(orc.level_density(level, p)), 0, math.pi / 2)
    assert abs(total - 1.0) < 1e-12
    for psi in (0.2, 0.7, 1.3):
        part, _ = integrate.quad(lambda p: float(orc.level_density(level, p)), 0, psi)
        assert abs(part - _cdf(level, psi)) < 1e-12
    mean, _ = integrate.quad(lambda p: p * float(orc.level_density(level, p)), 0, math.pi / 2)
    assert abs(mean - math.pi / 4) < 1e-12  # Lemma 1: E[Theta] = pi/4


def test_level2_variance_closed_form():
    var, _ = integrate.quad(lambda p: (p - math.pi / 4) ** 2 * float(orc.level_density(2, p)), 0, math.pi / 2)
    assert abs(var - (math.pi ** 2 / 16 - 0.5)) < 1e-12


def test_angles_of_gaussian_vectors_follow_lemma2():
    d = 128
    S = orc.make_rotation(d, seed=3)
    x = RNG.standard_normal((6000, d))
    angles, _ = orc.polar(orc.rotate(x, S), 4)
    assert stats.kstest(angles[0].ravel()[:100000], stats.uniform(0, 2 * math.pi).cdf).pvalue > 1e-3
    for level in (2, 3, 4):
        sample = angles[level - 1].ravel()[:60000]
        assert stats.kstest(sample, lambda p: _cdf(level, p)).pvalue > 1e-3
    # a wrong pairing (e.g. sine side first) would break levels >= 2 only through symmetry;
    # the level-1 quadrant convention is pinned by the worked example and the d=2 test.


# ---------------------------------------------------------------- codebooks (Eq. 4)
def test_level1_codebook_closed_form(cb):
    k = np.arange(16)
    assert np.allclose(cb.centroids[0], (2 * k + 1) * math.pi / 16, atol=1e-14)
    assert np.allclose(cb.boundaries[0], np.arange(1, 16) * math.pi / 8, atol=1e-14)


@pytest.mark.parametrize("level", [2, 3, 4])
def test_codebook_is_a_lloyd_max_fixed_point_by_independent_quadrature(cb, level):
    mpmath.mp.dps = 30
    theta, beta = cb.centroids[level - 1], cb.boundaries[level - 1]
    assert np.allclose(theta + theta[::-1], math.pi / 2, atol=1e-13)  # symmetric about pi/4
    assert abs(beta[1] - math.pi / 4) < 1e-14
    assert np.allclose(beta, 0.5 * (theta[:-1] + theta[1:]), atol=1e-15)
    k = 2 ** (level - 1)
    f = lambda p: mpmath.sin(2 * p) ** (k - 1)
    edges = [mpmath.mpf(0)] + [mpmath.mpf(float(b)) for b in beta] + [mpmath.pi / 2]
    for i in range(4):
        num = mpmath.quad(lambda p: p * f(p), [edges[i], edges[i + 1]])
        den = mpmath.quad(f, [edges[i], edges[i + 1]])
        assert abs(float(num / den) - theta[i]) < 1e-12


@pytest.mark.parametrize("level", [2, 3, 4])
def test_codebook_minimises_eq4_and_is_unique(cb, level):
    theta = cb.centroids[level - 1]

    def cost(c):
        b = np.concatenate(([0.0], 0.5 * (c[:-1] + c[1:]), [math.pi / 2]))
        return sum(integrate.quad(lambda p: (p - c[i]) ** 2 * float(orc.level_density(level, p)),
                                  b[i], b[i + 1])[0] for i in range(len(c)))

    base = cost(theta)
    for _ in range(20):
        assert cost(np.sort(theta + RNG.normal(0, 1e-3, 4))) > base
    skew, _ = orc.lloyd_max(level, 2, init=[0.05, 0.1, 0.2, 1.5])
    assert np.allclose(skew, theta, atol=1e-12)


def test_codebooks_match_the_tabulated_multiprecision_values(cb):
    """Centroids, outer boundaries and Eq. 4 cost of levels 2-4 against values tabulated from an independent
    40-digit computation (tests/golden/codebooks_levels_2_to_4.txt)."""
    rows = [ln.split() for ln in (GOLDEN / "codebooks_levels_2_to_4.txt").read_text().splitlines()
            if ln and not ln.startswith("#")]
    assert [int(r[0]) for r in rows] == [2, 3, 4]
    for r in rows:
        level, vals = int(r[0]), [float(v) for v in r[1:]]
        c, b = cb.centroids[level - 1], cb.boundaries[level - 1]
        assert np.allclose(c, vals[0:4], atol=1e-11, rtol=0)
        assert abs(b[0] - vals[4]) < 1e-11 and abs(b[1] - math.pi / 4) < 1e-13 and abs(b[2] - vals[5]) < 1e-11
        edges = np.concatenate(([0.0], b, [math.pi / 2]))
        k = 2 ** (level - 1)  # Lemma 2: Gamma(k) / (2^(k-2) Gamma(k/2)^2) sin^(k-1)(2 psi)
        const = math.gamma(k) / (2.0 ** (k - 2) * math.gamma(k / 2) ** 2)
        mse = sum(integrate.quad(lambda p: (p - c[i]) ** 2 * const * math.sin(2 * p) ** (k - 1), edges[i], edges[i + 1],
                                 epsabs=1e-14)[0] for i in range(4))
        assert abs(mse - vals[6]) < 2e-11


def test_level1_cost_closed_form(cb):
    # uniform density, 16 equal cells of width pi/8: mean squared error (pi/8)^2 / 12
    c = cb.centroids[0]
    b = np.concatenate(([0.0], cb.boundaries[0], [2 * math.pi]))
    mse = sum(integrate.quad(lambda p: (p - c[i]) ** 2 / (2 * math.pi), b[i], b[i + 1])[0] for i in range(16))
    assert abs(mse - (math.pi / 8) ** 2 / 12) < 1e-14


# ---------------------------------------------------------------- partial attentions
def test_merged_partial_attentions_equal_the_whole():
    """Eq. 2 with its sums split over disjoint token sets: any split, merged, gives the attention over all tokens;
    the log-sum-exp has its closed forms (one token: the score; n identical keys: score + log n; no token: -inf)."""
    rng = np.random.default_rng(8)
    d, n = 16, 50
    q, K, V = rng.normal(size=d), rng.normal(size=(n, d)) * 2, rng.normal(size=(n, d))
    whole = orc.softmax_attention(q, K, V, 0.3)
    assert abs(orc.log_sum_exp_scores(q, K[:1], 0.3) - 0.3 * K[0] @ q) < 1e-12
    same = np.repeat(K[:1], 7, axis=0)
    assert abs(orc.log_sum_exp_scores(q, same, 0.3) - (0.3 * K[0] @ q + math.log(7))) < 1e-12
    assert orc.log_sum_exp_scores(q, K[:0], 0.3) == -np.inf
    brute = math.log(sum(math.exp(0.3 * float(K[t] @ q)) for t in range(n)))
    assert abs(orc.log_sum_exp_scores(q, K, 0.3) - brute) < 1e-12
    for cuts in ([0, 50], [0, 1, 50], [0, 13, 13, 40, 50], [0, 0, 25, 50, 50]):      # empty sets included
        outs, lses = [], []
        for lo, hi in zip(cuts[:-1], cuts[1:]):
            outs.append(orc.softmax_attention(q, K[lo:hi], V[lo:hi], 0.3) if hi > lo else np.full(d, np.nan))
            lses.append(orc.log_sum_exp_scores(q, K[lo:hi], 0.3))
        out, lse = orc.merge_attention(np.array(outs), np.array(lses))
        assert np.allclose(out, whole, atol=1e-13) and abs(lse - brute) < 1e-12
    out, lse = orc.merge_attention(np.zeros((2, 3, d)), np.full((2, 3), -np.inf))
    assert np.all(out == 0) and np.all(lse == -np.inf)
    # scores far apart: the weights must not overflow
    out, lse = orc.merge_attention(np.array([np.ones(d), 3 * np.ones(d)]), np.array([800.0, -800.0]))
    assert np.allclose(out, 1.0) and lse == 800.0


def test_attention_with_an_unquantised_tail_is_attention_over_the_concatenation(cb):
    rng = np.random.default_rng(9)
    d, n, t = 16, 20, 6
    S = orc.make_rotation(d, 2)
    K, V = rng.normal(size=(n, d)), rng.normal(size=(n, d))
    kc, kr = orc.encode(K, S, cb)[:2]
    vc, vr = orc.encode(V, S, cb)[:2]
    q = rng.normal(size=(1, 2, d))
    kt, vt = rng.normal(size=(1, t, 1, d)), rng.normal(size=(1, t, 1, d))
    out, lse = orc.attention_with_tail(q, kc[None, None], kr[None, None], vc[None, None], vr[None, None], [n], cb, S, 0.25, kt, vt, [t])
    Kall = np.concatenate([orc.dequant(kc, kr, cb, S), kt[0, :, 0]])
    Vall = np.concatenate([orc.dequant(vc, vr, cb, S), vt[0, :, 0]])
    for h in range(2):
        s = Kall @ q[0, h] * 0.25
        p = np.exp(s - s.max())
        assert np.allclose(out[0, h], (p / p.sum()) @ Vall, atol=1e-13)
        assert abs(lse[0, h] - (s.max() + math.log(p.sum()))) < 1e-12
    # no tail: decode attention; no cache: exact attention over the tail
    a, _ = orc.attention_with_tail(q, kc[None, None], kr[None, None], vc[None, None], vr[None, None], [n], cb, S, 0.25, kt, vt, [0])
    assert np.allclose(a, orc.decode_attention(q, kc[None, None], kr[None, None], vc[None, None], vr[None, None], [n], cb, S, 0.25), atol=1e-13)
    b, _ = orc.attention_with_tail(q, kc[None, None], kr[None, None], vc[None, None], vr[None, None], [0], cb, S, 0.25, kt, vt, [t])
    for h in range(2):
        assert np.allclose(b[0, h], orc.softmax_attention(q[0, h], kt[0, :, 0], vt[0, :, 0], 0.25), atol=1e-13)


# ---------------------------------------------------------------- online codebook (Section 4.1)
def test_angle_histograms_count_every_angle_in_its_bin():
    S = np.eye(4)
    x = np.array([[3.0, 4.0, -8.0, 6.0], [1.0, 0.0, 0.0, -1.0]])     # level-1 angles: atan2(4,3), atan2(6,-8); 0, 3pi/2
    h = orc.angle_histograms(x, S, 2, 8)
    assert h.shape == (2, 8) and h[0].sum() == 4 and h[1].sum() == 2
    # bins of width pi/4: 0.927 -> 1, 2.498 -> 3, 0 -> 0, 3pi/2 -> 6
    assert h[0].tolist() == [1, 1, 0, 1, 0, 0, 1, 0]
    # level 2: atan2(10, 5) = 1.107 and atan2(1, 1) = pi/4, bins of width pi/16: 5 and 4
    assert h[1].tolist() == [0, 0, 0, 0, 1, 1, 0, 0]


def test_kmeans_on_histogram_fixed_point_toy_and_analytic_limit(cb):
    # two well separated clumps: the centroids are the clumps' weighted means, whatever the start
    counts = np.zeros(64)
    counts[[3, 4]] = [10, 30]
    counts[[40, 41, 42]] = [5, 5, 10]
    width = (math.pi / 2) / 64
    theta, beta = orc.kmeans_on_histogram(counts, 2, np.array([0.5, 0.6]))
    assert np.allclose(theta, [(10 * 3.5 + 30 * 4.5) / 40 * width, (5 * 40.5 + 5 * 41.5 + 10 * 42.5) / 20 * width], atol=1e-15)
    assert np.allclose(beta, [theta.mean()], atol=1e-15)
    # a histogram of the analytic density itself: the result is the analytic codebook up to the binning (each of
    # the n_c stationarity equations holds to half a bin, and the slack adds up along the chain of cells), it is a
    # fixed point (every centroid is the mean of its cell), and the discrete Eq. 4 cost does not exceed the start's
    for level in (1, 2, 4):
        n_bins, n_c = 4096, cb.centroids[level - 1].size
        hi = 2 * math.pi if level == 1 else math.pi / 2
        centres = (np.arange(n_bins) + 0.5) * hi / n_bins
        k = 2 ** (level - 1)
        dens = np.ones(n_bins) if level == 1 else np.sin(2 * centres) ** (k - 1)
        counts = np.round(dens / dens.sum() * 5e7)
        theta, beta = orc.kmeans_on_histogram(counts, level, cb.centroids[level - 1] + 0.01)
        assert theta.size == n_c and np.allclose(theta, cb.centroids[level - 1], atol=n_c * hi / n_bins)
        cell = np.searchsorted(beta, centres)
        for j in range(n_c):
            assert abs(theta[j] - np.average(centres[cell == j], weights=counts[cell == j])) < 1e-12
        cost = lambda t: np.sum(counts * np.min((centres[:, None] - t[None, :]) ** 2, axis=1))
        assert cost(theta) <= cost(cb.centroids[level - 1] + 0.01)


def test_online_codebook_follows_the_data():
    """Gaussian data give back (nearly) the analytic codebook; data that are not isotropic after the rotation move
    it, and the fitted codebook then encodes those data with a smaller error than the analytic one."""
    rng = np.random.default_rng(12)
    d = 16
    S = orc.make_rotation(d, 1)
    offline = orc.fit_codebooks()
    x = rng.normal(size=(20000, d))
    online = orc.fit_codebooks_online(x, S)
    for level in range(4):
        # level 1: 16 cells of width 0.39 on a flat density, where sampling noise moves the optimum most
        assert np.allclose(online.centroids[level], offline.centroids[level], atol=0.08 if level == 0 else 0.02)
    skew = x * np.linspace(0.2, 3.0, d)[None, :] @ S.T        # anisotropic in the rotated basis
    online = orc.fit_codebooks_online(skew, S)
    err = lambda cbk: np.mean(np.sum((orc.dequant(*orc.encode(skew, S, cbk)[:2], cbk, S) - skew) ** 2, axis=1))
    assert err(online) < 0.97 * err(offline)


# ---------------------------------------------------------------- radii (b_FPN = 16)
def test_radius_rounding_is_round_to_nearest_even_and_saturates():
    """binary16 spacing in [1, 2) is 2^-10: a value 3/4 of the way up rounds up (truncation would not), exact ties
    go to the even significand, 65504 is the largest finite value; anything above it saturates and is counted."""
    ulp = 2.0 ** -10
    r16, sat = orc.round_radii_fp16(np.array([1 + 0.75 * ulp, 1 + 0.5 * ulp, 1 + 1.5 * ulp, 1 + 0.25 * ulp, 2048.0 + 1.0,
                                              2048.0 + 3.0, 65504.0, 0.0]))
    assert sat == 0
    assert r16.dtype == np.float16
    assert r16.astype(np.float64).tolist() == [1 + ulp, 1.0, 1 + 2 * ulp, 1.0, 2048.0, 2052.0, 65504.0, 0.0]
    r16, sat = orc.round_radii_fp16(np.array([70000.0, 65504.0, 65519.0, 1e9, 3.0]))
    assert sat == 3 and r16.astype(np.float64).tolist() == [65504.0, 65504.0, 65504.0, 65504.0, 3.0]


# ---------------------------------------------------------------- Quant
def test_boundary_count_equals_printed_argmin(cb):
    for l in range(4):
        hi = 2 * math.pi if l == 0 else math.pi / 2
        psi = RNG.uniform(0, hi, 20000)
        adv = np.concatenate([np.nextafter(cb.boundaries[l], -np.inf), np.nextafter(cb.boundaries[l], np.inf),
                              np.nextafter(np.nextafter(cb.boundaries[l], np.inf), np.inf),
                              cb.centroids[l], [0.0, hi]])
        for p in (psi, adv):
            a = orc.quantize_angles(p, cb.boundaries[l])
            b = orc.quantize_angles_argmin(p, cb.centroids[l])
            diff = a != b
            # the two rules may only differ where the two distances tie to rounding
            if diff.any():
                d0 = np.abs(p[diff] - cb.centroids[l][a[diff]])
                d1 = np.abs(p[diff] - cb.centroids[l][b[diff]])
                assert np.all(np.abs(d0 - d1) < 1e-15)
        assert orc.quantize_angles(psi, cb.boundaries[l]).max() == 2 ** cb.bits[l] - 1


def test_worked_example_d4():
    rows = {}
    for line in (GOLDEN / "worked_example_d4.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            key, *vals = line.split()
            rows[key] = np.array([float(v) for v in vals])
    c1, b1 = orc.lloyd_max(1, 4)
    c2, b2 = orc.lloyd_max(2, 2)
    cbk = orc.Codebooks((4, 2), (c1, c2), (b1, b2))
    codes, radii16, angles = orc.encode(rows["y"][None], np.eye(4), cbk)
    assert np.allclose(angles[0][0], rows["level1_angles"], atol=1e-15)
    assert np.allclose(angles[1][0], rows["level2_angle"], atol=1e-15)
    assert list(codes[0]) == [int(v) for v in np.concatenate([rows["level1_codes"], rows["level2_code"]])]
    assert float(radii16[0, 0]) == rows["radius_fp16"][0]
    # hand-computed DeQuant of the same codes
    t2 = c2[3]
    r1 = 11.1796875 * np.array([math.cos(t2), math.sin(t2)])
    expect = np.array([r1[0] * math.cos(5 * math.pi / 16), r1[0] * math.sin(5 * math.pi / 16),
                       r1[1] * math.cos(13 * math.pi / 16), r1[1] * math.sin(13 * math.pi / 16)])
    got = orc.dequant(codes, radii16, cbk, np.eye(4))[0]
    assert np.allclose(got, expect, atol=1e-14)
    assert got[2] < 0 < got[3]  # second pair sits in the second quadrant


def test_bit_budget_of_section_4_1(cb):
    d = 128
    x = RNG.standard_normal((3, d))
    codes, radii16, _ = orc.encode(x, np.eye(d), cb)
    assert codes.shape == (3, 120) and radii16.shape == (3, 8) and radii16.dtype == np.float16
    per_level = orc.split_codes(codes, d, 4)
    bits = sum(per_level[l].shape[-1] * cb.bits[l] for l in range(4)) + 16 * radii16.shape[-1]
    assert bits == 8 * 62 and bits / d == 3.875  # 62 bits per 16 coordinates


# ---------------------------------------------------------------- brute force on tiny vectors
def _all_codewords(cbk, d):
    """Every reconstructable unit-radius direction for a full log2(d)-level transform."""
    levels = len(cbk.bits)
    counts = [d >> (l + 1) for l in range(levels)]
    grids = [itertools.product(range(2 ** cbk.bits[l]), repeat=counts[l]) for l in range(levels)]
    for combo in itertools.product(*grids):
        yield np.concatenate([np.array(c, dtype=np.uint8) for c in combo])


def test_bruteforce_d4_greedy_vs_global():
    c1, b1 = orc.lloyd_max(1, 4)
    c2, b2 = orc.lloyd_max(2, 2)
    cbk = orc.Codebooks((4, 2), (c1, c2), (b1, b2))
    words = np.array(list(_all_codewords(cbk, 4)))  # 16*16*4 = 1024
    assert len(words) == 1024
    dirs = orc.dequant_rotated(words, np.ones((len(words), 1), np.float16), cbk, 4)
    assert np.allclose(np.linalg.norm(dirs, axis=1), 1.0, atol=1e-14)
    x = RNG.standard_normal((400, 4))
    codes, _, _ = orc.encode(x, np.eye(4), cbk)
    u = x / np.linalg.norm(x, axis=1, keepdims=True)
    sims = u @ dirs.T
    best = np.argmax(sims, axis=1)
    greedy_sim = np.array([sims[i, np.flatnonzero((words == codes[i]).all(1))[0]] for i in range(len(x))])
    assert np.all(greedy_sim <= sims[np.arange(len(x)), best] + 1e-15)  # never better than the optimum
    # (i) level-1 greedy codes are globally optimal once the top code is fixed to the optimum's
    assert np.array_equal(words[best][:, :2], codes[:, :2])
    # greedy equals the optimum for the large majority, but not always (per-angle rounding)
    agree = np.mean((words[best] == codes).all(1))
    assert 0.95 < agree <= 1.0


def test_bruteforce_d16_per_level_optimality(cb):
    """With every other code held at its greedy value, the greedy level-1 code of each pair is
    the best of the 16 candidates (the reconstruction's inner product is a non-negative
    combination of cos(level-1 angle errors))."""
    d = 16
    x = RNG.standard_normal((40, d))
    codes, radii16, _ = orc.encode(x, np.eye(d), cb)
    for i in range(len(x)):
        for j in range(8):
            trial = np.repeat(codes[i][None], 16, axis=0)
            trial[:, j] = np.arange(16)
            rec = orc.dequant_rotated(trial, np.repeat(radii16[i][None], 16, 0), cb, d)
            assert int(np.argmax(rec @ x[i])) == int(codes[i, j])


def test_expected_distortion_matches_closed_form(cb):
    """Independence of the angles (Lemma 2) gives E||x-x_hat||^2/||x||^2 = 2 - 2 prod_l E[cos(err_l)]
    when the radius is kept; the per-level factors come from quadrature of the density."""
    prod = 1.0
    for l in range(4):
        hi = 2 * math.pi if l == 0 else math.pi / 2
        edges = np.concatenate(([0.0], cb.boundaries[l], [hi]))
        e = sum(integrate.quad(lambda p: math.cos(p - cb.centroids[l][k]) * float(orc.level_density(l + 1, p)),
                               edges[k], edges[k + 1])[0] for k in range(len(edges) - 1))
        prod *= e
    expect = 2 - 2 * prod
    assert abs(expect - 0.0320765) < 2e-6
    d = 128
    S = orc.make_rotation(d, 11)
    rel = []
    for scale in (1.0, 37.0):  # Theorem 1: relative error does not depend on ||x||
        x = RNG.standard_normal((20000, d)) * scale
        codes, radii16, _ = orc.encode(x, S, cb)
        xh = orc.dequant(codes, radii16, cb, S)
        rel.append(np.mean(np.sum((x - xh) ** 2, 1) / np.sum(x * x, 1)))
    assert abs(rel[0] - expect) < 4e-4 and abs(rel[1] - expect) < 4e-4


# ---------------------------------------------------------------- attention (Eq. 3)
def _small_cache(cb, B=2, Hkv=2, n=37, d=16, seed=5):
    S = orc.make_rotation(d, seed)
    cache = orc.OracleCache(B, Hkv, n + 4, d, cb, S)
    rng = np.random.default_rng(seed)
    for b in range(B):
        cache.encode_chunk(b, rng.standard_normal((n - b, Hkv, d)), rng.standard_normal((n - b, Hkv, d)))
    return cache, S, rng


def test_attention_len1_returns_the_dequantised_value(cb):
    d = 16
    S = orc.make_rotation(d, 1)
    cache = orc.OracleCache(1, 1, 4, d, cb, S)
    k, v = RNG.standard_normal((1, 1, d)), RNG.standard_normal((1, 1, d))
    cache.encode_chunk(0, k, v)
    out = cache.attend(RNG.standard_normal((1, 2, d)), 0.25)
    vhat = orc.dequant(cache.v_codes[0, 0, :1], cache.v_radii[0, 0, :1], cb, S)[0]
    assert np.allclose(out[0, 0], vhat, atol=1e-15) and np.allclose(out[0, 1], vhat, atol=1e-15)


def test_attention_identical_keys_average_the_values(cb):
    d = 16
    S = orc.make_rotation(d, 2)
    cache = orc.OracleCache(1, 1, 8, d, cb, S)
    k = np.repeat(RNG.standard_normal((1, 1, d)), 8, axis=0)
    v = RNG.standard_normal((8, 1, d))
    cache.encode_chunk(0, k, v)
    out = cache.attend(RNG.standard_normal((1, 1, d)), 0.25)
    vhat = orc.dequant(cache.v_codes[0, 0], cache.v_radii[0, 0], cb, S)
    assert np.allclose(out[0, 0], vhat.mean(0), atol=1e-14)


def test_attention_equals_rotated_basis_evaluation_and_gqa_mapping(cb):
    cache, S, rng = _small_cache(cb)
    B, Hkv, d, Hq = 2, 2, 16, 4
    q = rng.standard_normal((B, Hq, d))
    out = cache.attend(q, 0.25)
    for b in range(B):
        n = int(cache.lens[b])
        for h in range(Hq):
            hk = h // 2
            yk = orc.dequant_rotated(cache.k_codes[b, hk, :n], cache.k_radii[b, hk, :n], cb, d)
            yv = orc.dequant_rotated(cache.v_codes[b, hk, :n], cache.v_radii[b, hk, :n], cb, d)
            s = yk @ (q[b, h] @ S) * 0.25  # <q, y S^T> = <q S, y>
            p = special.softmax(s)
            assert np.allclose(out[b, h], (p @ yv) @ S.T, atol=1e-13)


def test_exact_attention_special_cases_and_brute_force():
    """Eq. 2 on the unquantised cache (reported as information only): one token returns its value, identical keys
    average the values, and a small case equals the definition written out with Python loops."""
    rng = np.random.default_rng(3)
    B, Hq, Hkv, n, d = 2, 4, 2, 5, 8
    K, V, q = rng.normal(size=(B, Hkv, n, d)), rng.normal(size=(B, Hkv, n, d)), rng.normal(size=(B, Hq, d))
    one = orc.exact_attention(q, K, V, [1, 1], 0.3)
    for h in range(Hq):
        assert np.allclose(one[:, h], V[:, h // 2, 0], atol=1e-15)
    same = orc.exact_attention(q, np.repeat(K[:, :, :1], n, axis=2), V, [n, n], 0.3)
    for h in range(Hq):
        assert np.allclose(same[:, h], V[:, h // 2].mean(axis=1), atol=1e-14)
    got = orc.exact_attention(q, K, V, [n, 3], 0.3)
    for b, nb in enumerate([n, 3]):
        for h in range(Hq):
            w = [math.exp(0.3 * sum(q[b, h, i] * K[b, h // 2, t, i] for i in range(d))) for t in range(nb)]
            want = [sum(w[t] * V[b, h // 2, t, i] for t in range(nb)) / sum(w) for i in range(d)]
            assert np.allclose(got[b, h], want, atol=1e-13)


def test_multi_query_attention_is_the_causal_stream(cb):
    """The chunk of n_q queries at the end of a sequence: one query reduces to decode attention; in general the
    result equals a masked softmax over all cached tokens (scores of the tokens a query must not see set to -inf),
    written here with explicit loops on the dequantised cache."""
    rng = np.random.default_rng(9)
    B, Hq, Hkv, d, n_q = 2, 4, 2, 16, 3
    S = orc.make_rotation(d, 4)
    cache = orc.OracleCache(B, Hkv, 12, d, cb, S)
    for b, n in enumerate((9, 2)):
        cache.encode_chunk(b, rng.normal(size=(n, Hkv, d)), rng.normal(size=(n, Hkv, d)))
    q = rng.normal(size=(B, n_q, Hq, d))
    args = (cache.k_codes, cache.k_radii, cache.v_codes, cache.v_radii, cache.lens, cb, S, 0.3)
    got = orc.multi_query_attention(q, *args)
    assert np.allclose(orc.multi_query_attention(q[:, -1:], *args)[:, 0], orc.decode_attention(q[:, -1], *args), atol=1e-15)
    for b in range(B):
        n = int(cache.lens[b])
        for h in range(Hq):
            K = orc.dequant(cache.k_codes[b, h // 2, :n], cache.k_radii[b, h // 2, :n], cb, S)
            V = orc.dequant(cache.v_codes[b, h // 2, :n], cache.v_radii[b, h // 2, :n], cb, S)
            for j in range(n_q):
                last_visible = n - n_q + j           # position of the query's own token
                w = [math.exp(0.3 * float(K[t] @ q[b, j, h])) if t <= last_visible else 0.0 for t in range(n)]
                want = sum(w[t] * V[t] for t in range(n)) / sum(w) if sum(w) > 0 else np.zeros(d)
                assert np.allclose(got[b, j, h], want, atol=1e-13)
    assert np.all(got[1, 0] == 0)  # sequence 1 holds 2 tokens: the first of 3 queries precedes them all


def test_attention_without_quantisation_does_not_depend_on_S():
    d, n = 16, 50
    K, V, q = RNG.standard_normal((n, d)), RNG.standard_normal((n, d)), RNG.standard_normal(d)
    ref = special.softmax(K @ q * 0.25) @ V
    for seed in (1, 2):
        S = orc.make_rotation(d, seed)
        ak, rk = orc.polar(orc.rotate(K, S), 4)
        av, rv = orc.polar(orc.rotate(V, S), 4)
        Kb, Vb = orc.inverse_polar(ak, rk) @ S.T, orc.inverse_polar(av, rv) @ S.T
        assert np.allclose(orc.softmax_attention(q, Kb, Vb, 0.25), ref, atol=1e-12)


def test_chunked_encode_and_append_match_one_shot(cb):
    d, Hkv, n = 16, 2, 23
    S = orc.make_rotation(d, 9)
    K, V = RNG.standard_normal((n, Hkv, d)), RNG.standard_normal((n, Hkv, d))
    one = orc.OracleCache(1, Hkv, 32, d, cb, S)
    one.encode_chunk(0, K, V)
    two = orc.OracleCache(1, Hkv, 32, d, cb, S)
    two.encode_chunk(0, K[:10], V[:10])
    two.encode_chunk(0, K[10:22], V[10:22])
    two.append(K[22][None], V[22][None])
    assert two.lens[0] == n
    for name in ("k_codes", "v_codes", "k_radii", "v_radii"):
        assert np.array_equal(getattr(one, name), getattr(two, name))


def test_boundary_distance_accounting(cb):
    psi = [np.array([[1e-7, math.pi / 8 + 2e-7, 6.0]]), np.array([[math.pi / 4 - 3e-7]])]
    cbk = orc.Codebooks((4, 2), cb.centroids[:2], cb.boundaries[:2])
    dist = orc.boundary_distance(psi, cbk)
    assert np.allclose(dist[0, :2], [1e-7, 2e-7], atol=1e-12) and dist[0, 2] > 0.1
    assert abs(dist[0, 3] - 3e-7) < 1e-12
