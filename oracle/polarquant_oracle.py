"""Float64 CPU oracle for the PolarQuant hot path (KV-cache encode + decode attention).

THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the tests, the smoke check and
the benchmark's CPU-baseline / reference legs may import it.  It shares nothing with
the CUDA path: no tables, no constants, no helpers.  It is written to be checked
against the paper by eye, not to be fast: every function follows one passage of the
paper, step by step, in float64, vectorised over tokens only (no tiling, no fusion,
no reordering of the method's steps).

Conventions (the paper is 1-indexed, this file is 0-indexed):

* Row-vector form of Algorithm 1: ``y = x @ S`` and ``x_hat = y_hat @ S.T``.
* A level-l angle with index j is computed from entries ``2j`` (the cosine side) and
  ``2j+1`` (the sine side) of the level-(l-1) radius vector; level 0 is ``y`` itself.
* The recursion runs for ``L`` levels (Section 4.1 uses L = 4), so a d-vector becomes
  ``d / 2**L`` radii plus ``d/2 + d/4 + ... + d/2**L`` angles.
* Canonical code order of one vector: all level-1 codes (j = 0 .. d/2-1), then all
  level-2 codes, ... then level-L codes.  Radii follow in index order.
* Level 1 angles live in [0, 2*pi), higher levels in [0, pi/2] (Definition 1).

Pins (tests/test_oracle_*.py): exact invertibility of the unquantised transform,
block radius == block norm, norm preservation under S, the structured preconditioners against the closed form of
the Sylvester matrix and the fast Walsh-Hadamard butterfly, Lemma 2 densities against the
incomplete-beta CDF, Lloyd-Max fixed-point equations against independent quadrature,
the worked d=4 example under tests/golden/, brute force on d=4 and d=16, closed-form
expected distortion, the len=1 / identical-keys attention special cases, multi-query attention against a
masked softmax, merging of partial attentions (a split of the tokens gives back the whole; closed forms of the
log-sum-exp), and the online codebook (histogram counts, k-means fixed point, two-cluster toy, convergence to the
analytic codebook on samples of the analytic density).
Parity unpinned: nothing in this file; quality on real model caches is out of scope.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

TWO_PI = 2.0 * math.pi
HALF_PI = 0.5 * math.pi

DEFAULT_BITS = (4, 2, 2, 2)  # Section 4.1: 4 bits at level 1, 2 bits at levels 2..4


# --------------------------------------------------------------------------------------
# Random preconditioning (Section 3.2 footnote, Section 4.1: "a random rotational matrix")
# --------------------------------------------------------------------------------------
def make_rotation(d: int, seed: int) -> np.ndarray:
    """Haar-distributed orthogonal d x d matrix: QR of a seeded Gaussian, with the
    signs of R's diagonal folded into Q so that the distribution is uniform."""
    rng = np.random.default_rng(seed)
    g = rng.standard_normal((d, d))
    q, r = np.linalg.qr(g)
    sign = np.where(np.diag(r) < 0.0, -1.0, 1.0)
    return q * sign[None, :]


def make_structured_rotation(d: int, kind: str, signs=None) -> np.ndarray:
    """Preconditioners without a dense random matrix.  Section 3.2 only asks for an orthogonal S that spreads a vector
    over its coordinates (the footnote's fast transforms), and Section 5's rows named "PolarQuant" (without "-R") use
    none at all.  kind "identity": S = I.  kind "hadamard": S = diag(signs) H_d / sqrt(d), with H_d the Sylvester
    Hadamard matrix of a power-of-two order, H_1 = [1], H_2n = [[H_n, H_n], [H_n, -H_n]], and signs in {+1, -1}
    drawn by the caller (y = x . S flips the signs of x, then transforms)."""
    if kind == "identity":
        return np.eye(d, dtype=np.float64)
    if kind != "hadamard" or d < 1 or d & (d - 1):
        raise ValueError("kind must be 'identity' or 'hadamard' (power-of-two order)")
    H = np.ones((1, 1), dtype=np.float64)
    while H.shape[0] < d:
        H = np.block([[H, H], [H, -H]])
    sg = np.asarray(signs, dtype=np.float64)
    if sg.shape != (d,) or not np.all(np.abs(sg) == 1.0):
        raise ValueError("signs must be d entries of +1 or -1")
    return sg[:, None] * H / np.sqrt(float(d))


def rotate(x: np.ndarray, S: np.ndarray) -> np.ndarray:
    """Algorithm 1 line 2: y_i = x_i . S for every row."""
    return np.asarray(x, dtype=np.float64) @ np.asarray(S, dtype=np.float64)


# --------------------------------------------------------------------------------------
# Recursive polar transform (Definition 1, procedure Polar of Algorithm 1)
# --------------------------------------------------------------------------------------
def polar(y: np.ndarray, n_levels: int):
    """Polar(y) for every row of ``y`` (shape [..., d]).

    Returns ``(angles, radii)`` where ``angles[l-1]`` has shape [..., d / 2**l] and
    ``radii`` (the level-L radius vector) has shape [..., d / 2**L].
    """
    r = np.asarray(y, dtype=np.float64)
    angles = []
    for level in range(1, n_levels + 1):
        a = r[..., 0::2]  # entries 2j   : cosine side
        b = r[..., 1::2]  # entries 2j+1 : sine side
        psi = np.arctan2(b, a)
        if level == 1:
            # Level 1 covers the full circle [0, 2*pi); arctan2 returns (-pi, pi].
            psi = np.where(psi < 0.0, psi + TWO_PI, psi)
        psi = psi + 0.0  # turns -0.0 into +0.0
        angles.append(psi)
        r = np.hypot(a, b)
    return angles, r


def inverse_polar(angles, radii: np.ndarray) -> np.ndarray:
    """The reverse map of Definition 1 in the form procedure DeQuant states it:
    from the top level down, r[2j] = r_parent[j] cos(psi_j), r[2j+1] = r_parent[j] sin(psi_j)."""
    r = np.asarray(radii, dtype=np.float64)
    for psi in reversed(list(angles)):
        child = np.empty(r.shape[:-1] + (2 * r.shape[-1],), dtype=np.float64)
        child[..., 0::2] = r * np.cos(psi)
        child[..., 1::2] = r * np.sin(psi)
        r = child
    return r


# --------------------------------------------------------------------------------------
# Angle densities (Lemma 2) and codebooks (Eq. 4)
# --------------------------------------------------------------------------------------
def level_density(level: int, psi):
    """Marginal density of one level-``level`` angle of an isotropic Gaussian vector."""
    psi = np.asarray(psi, dtype=np.float64)
    if level == 1:
        return np.full_like(psi, 1.0 / TWO_PI)
    k = 2 ** (level - 1)  # the two child radii are norms of k-dimensional Gaussians
    const = math.gamma(k) / (2.0 ** (k - 2) * math.gamma(k / 2.0) ** 2)
    return const * np.sin(2.0 * psi) ** (k - 1)


@dataclass(frozen=True)
class Codebooks:
    """Per level: ``centroids[l]`` (2**b_l ascending angles) and ``boundaries[l]``
    (the 2**b_l - 1 interior cell boundaries)."""
    bits: tuple
    centroids: tuple
    boundaries: tuple

    @property
    def n_levels(self) -> int:
        return len(self.bits)

    def flat_centroids(self) -> np.ndarray:
        return np.concatenate(self.centroids)

    def flat_boundaries(self) -> np.ndarray:
        return np.concatenate(self.boundaries)


_GL_X, _GL_W = np.polynomial.legendre.leggauss(96)


def _integrate(fn, lo: float, hi: float) -> float:
    """Gauss-Legendre quadrature of a smooth function on [lo, hi]."""
    half = 0.5 * (hi - lo)
    mid = 0.5 * (hi + lo)
    return float(half * np.sum(_GL_W * fn(mid + half * _GL_X)))


def lloyd_max(level: int, n_bits: int, init=None, tol: float = 1e-15, max_iter: int = 100000):
    """Minimiser of Eq. 4 for one level: alternate (boundaries = midpoints of adjacent
    centroids) and (centroid = conditional mean of the density on its cell) to a fixed
    point.  Returns (centroids, interior boundaries)."""
    n = 2 ** n_bits
    lo, hi = (0.0, TWO_PI) if level == 1 else (0.0, HALF_PI)
    if init is None:
        theta = lo + (np.arange(n) + 0.5) * (hi - lo) / n
    else:
        theta = np.array(init, dtype=np.float64)
    dens = lambda p: level_density(level, p)
    mom = lambda p: p * level_density(level, p)
    for _ in range(max_iter):
        beta = 0.5 * (theta[:-1] + theta[1:])
        edges = np.concatenate(([lo], beta, [hi]))
        new = np.array([
            _integrate(mom, edges[k], edges[k + 1]) / _integrate(dens, edges[k], edges[k + 1])
            for k in range(n)
        ])
        delta = float(np.max(np.abs(new - theta)))
        theta = new
        if delta < tol:
            break
    beta = 0.5 * (theta[:-1] + theta[1:])
    return theta, beta


def fit_codebooks(bits=DEFAULT_BITS) -> Codebooks:
    """Algorithm 1 line 3 with the analytic densities of Lemma 2 ("offline" codebook)."""
    cents, bounds = [], []
    for level, b in enumerate(bits, start=1):
        c, t = lloyd_max(level, b)
        cents.append(c)
        bounds.append(t)
    return Codebooks(tuple(bits), tuple(cents), tuple(bounds))


# --------------------------------------------------------------------------------------
# "Online" codebook (Section 4.1): clustering of the observed angles of one prompt and layer
# --------------------------------------------------------------------------------------
def angle_histograms(x: np.ndarray, S: np.ndarray, n_levels: int, n_bins: int) -> np.ndarray:
    """The angles that Polar (Algorithm 1) produces for the rows of ``x`` ([n, d]; keys and values of the
    prompt stacked), counted per level in ``n_bins`` bins of equal width over the level's range ([0, 2 pi) at level
    1, [0, pi/2] above).  The histogram is the sample the clustering runs on: an angle stands for the centre of
    its bin.  Returns int64 [n_levels, n_bins]."""
    angles, _ = polar(rotate(x, S), n_levels)
    hist = np.zeros((n_levels, n_bins), dtype=np.int64)
    for level in range(1, n_levels + 1):
        width = (TWO_PI if level == 1 else HALF_PI) / n_bins
        idx = np.minimum((angles[level - 1].ravel() / width).astype(np.int64), n_bins - 1)
        hist[level - 1] = np.bincount(idx, minlength=n_bins)
    return hist


def kmeans_on_histogram(counts: np.ndarray, level: int, init: np.ndarray, max_iter: int = 10000):
    """1-D k-means (Lloyd's iteration) on binned samples: the discrete form of Eq. 4, with the bin centres as
    sample values and the counts as weights.  Alternates (cell boundaries = midpoints of adjacent centroids) and
    (centroid = weighted mean of the bin centres in its cell; an empty cell keeps its centroid) until nothing moves.
    k-means++ in the paper is a randomised choice of the starting centroids; this reading starts from ``init``
    (the analytic codebook of the level), which makes the result a function of the data alone.  Distances are taken
    on the line, also at level 1, as Quant is printed.  Returns (centroids, interior boundaries)."""
    counts = np.asarray(counts, dtype=np.float64)
    n_bins = counts.size
    width = (TWO_PI if level == 1 else HALF_PI) / n_bins
    centres = (np.arange(n_bins) + 0.5) * width
    theta = np.array(init, dtype=np.float64)
    for _ in range(max_iter):
        beta = 0.5 * (theta[:-1] + theta[1:])
        cell = np.searchsorted(beta, centres, side="left")      # number of boundaries below the bin centre
        new = theta.copy()
        for k in range(theta.size):
            w = counts[cell == k]
            if w.sum() > 0:
                new[k] = float(np.sum(w * centres[cell == k]) / w.sum())
        if np.array_equal(new, theta):
            break
        theta = new
    return theta, 0.5 * (theta[:-1] + theta[1:])


def fit_codebooks_online(x: np.ndarray, S: np.ndarray, bits=DEFAULT_BITS, n_bins: int = 4096) -> Codebooks:
    """Algorithm 1 line 3 with the "online" codebook of Section 4.1: per level, k-means on the observed angles of
    this input (binned), started from the analytic codebook."""
    offline = fit_codebooks(bits)
    hist = angle_histograms(x, S, len(bits), n_bins)
    cents, bounds = [], []
    for level in range(1, len(bits) + 1):
        c, t = kmeans_on_histogram(hist[level - 1], level, offline.centroids[level - 1])
        cents.append(c)
        bounds.append(t)
    return Codebooks(tuple(bits), tuple(cents), tuple(bounds))


def codebooks_from_arrays(bits, flat_centroids, flat_boundaries=None) -> Codebooks:
    """Wrap externally supplied centroids (float64, ascending per level).  Boundaries
    default to the midpoints of adjacent centroids (nearest-centroid rule)."""
    flat_centroids = np.asarray(flat_centroids, dtype=np.float64)
    cents, bounds, pos, bpos = [], [], 0, 0
    for b in bits:
        n = 2 ** b
        c = flat_centroids[pos:pos + n].copy()
        pos += n
        if flat_boundaries is None:
            t = 0.5 * (c[:-1] + c[1:])
        else:
            t = np.asarray(flat_boundaries, dtype=np.float64)[bpos:bpos + n - 1].copy()
            bpos += n - 1
        cents.append(c)
        bounds.append(t)
    return Codebooks(tuple(bits), tuple(cents), tuple(bounds))


# --------------------------------------------------------------------------------------
# Quant / DeQuant (Algorithm 1)
# --------------------------------------------------------------------------------------
def quantize_angles(psi: np.ndarray, boundaries: np.ndarray) -> np.ndarray:
    """Procedure Quant: index of the nearest centroid.  With boundaries at the midpoints
    this is the number of interior boundaries strictly below psi (ties go to the lower
    index; distance on the line, not on the circle)."""
    psi = np.asarray(psi, dtype=np.float64)
    return np.sum(psi[..., None] > boundaries, axis=-1).astype(np.uint8)


def quantize_angles_argmin(psi: np.ndarray, centroids: np.ndarray) -> np.ndarray:
    """Procedure Quant exactly as printed: argmin_k |theta_k - psi| (first minimum)."""
    psi = np.asarray(psi, dtype=np.float64)
    return np.argmin(np.abs(psi[..., None] - centroids), axis=-1).astype(np.uint8)


def round_radii_fp16(radii: np.ndarray):
    """b_FPN = 16: one rounding float64 -> binary16, round-to-nearest-even, saturating
    at the largest finite value.  Returns (fp16 array, number saturated)."""
    r = np.asarray(radii, dtype=np.float64)
    sat = r > 65504.0
    r16 = np.where(sat, 65504.0, r).astype(np.float16)
    return r16, int(np.count_nonzero(sat))


def encode(x: np.ndarray, S: np.ndarray, cb: Codebooks):
    """PolarQuant (Algorithm 1 lines 2 and 4) for rows of ``x`` ([..., d]).

    Returns ``(codes, radii16, angles)``: uint8 codes in canonical order
    [..., sum_l d/2**l], float16 radii [..., d/2**L], and the unquantised float64
    angles per level (for boundary-distance accounting in the parity tests)."""
    y = rotate(x, S)
    angles, radii = polar(y, cb.n_levels)
    codes = [quantize_angles(angles[l], cb.boundaries[l]) for l in range(cb.n_levels)]
    radii16, _ = round_radii_fp16(radii)
    return np.concatenate(codes, axis=-1), radii16, angles


def split_codes(codes: np.ndarray, d: int, n_levels: int):
    """Canonical code vector -> list of per-level code arrays."""
    out, pos = [], 0
    for level in range(1, n_levels + 1):
        n = d >> level
        out.append(codes[..., pos:pos + n])
        pos += n
    return out


def dequant_rotated(codes: np.ndarray, radii16: np.ndarray, cb: Codebooks, d: int) -> np.ndarray:
    """Procedure DeQuant without the final multiplication by S^T (the rotated basis)."""
    per_level = split_codes(np.asarray(codes), d, cb.n_levels)
    angles = [cb.centroids[l][per_level[l].astype(np.int64)] for l in range(cb.n_levels)]
    return inverse_polar(angles, np.asarray(radii16).astype(np.float64))


def dequant(codes, radii16, cb: Codebooks, S: np.ndarray) -> np.ndarray:
    """Procedure DeQuant: centroid angles + stored radii -> r^(0) . S^T."""
    d = S.shape[0]
    return dequant_rotated(codes, radii16, cb, d) @ np.asarray(S, dtype=np.float64).T


# --------------------------------------------------------------------------------------
# Attention over the dequantised cache (Eq. 2 / Eq. 3)
# --------------------------------------------------------------------------------------
def softmax_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """softmax(K q * scale)^T V for one query ``q`` [d], keys/values [n, d]."""
    s = (K @ q) * scale
    s = s - np.max(s)
    p = np.exp(s)
    p = p / np.sum(p)
    return p @ V


def decode_attention(q, k_codes, k_radii, v_codes, v_radii, lens, cb: Codebooks, S, scale):
    """Eq. 3 for a batch: one query per (sequence, query head).

    q        [B, Hq, d]                     float64-convertible
    *_codes  [B, Hkv, capacity, n_codes]    uint8, canonical order
    *_radii  [B, Hkv, capacity, d/2**L]     float16
    lens     [B]                            cached tokens per sequence
    Query head h reads kv-head h // (Hq // Hkv).  Returns float64 [B, Hq, d].
    """
    q = np.asarray(q, dtype=np.float64)
    B, Hq, d = q.shape
    Hkv = k_codes.shape[1]
    group = Hq // Hkv
    out = np.zeros((B, Hq, d), dtype=np.float64)
    for b in range(B):
        n = int(lens[b])
        for hk in range(Hkv):
            K_hat = dequant(k_codes[b, hk, :n], k_radii[b, hk, :n], cb, S)
            V_hat = dequant(v_codes[b, hk, :n], v_radii[b, hk, :n], cb, S)
            for h in range(hk * group, (hk + 1) * group):
                out[b, h] = softmax_attention(q[b, h], K_hat, V_hat, scale)
    return out


def multi_query_attention(q, k_codes, k_radii, v_codes, v_radii, lens, cb: Codebooks, S, scale):
    """Eq. 2 / Eq. 3 for the last ``n_q`` positions of every sequence at once (a chunk of a prefill, or the
    drafted tokens of a speculative step): in the stream of Section 4 the i-th query attends to the first i
    tokens, so query ``j`` (0-based) of the chunk sees the cached tokens ``t < lens[b] - (n_q - 1 - j)``; the
    last query sees all of them.  The keys and values of the chunk itself are already in the cache.

    q  [B, n_q, Hq, d];  the other arguments as in decode_attention.  Returns float64 [B, n_q, Hq, d]
    (a query that would see no token returns zeros).
    """
    q = np.asarray(q, dtype=np.float64)
    B, n_q, Hq, d = q.shape
    Hkv = k_codes.shape[1]
    group = Hq // Hkv
    out = np.zeros((B, n_q, Hq, d), dtype=np.float64)
    for b in range(B):
        n = int(lens[b])
        for hk in range(Hkv):
            K_hat = dequant(k_codes[b, hk, :n], k_radii[b, hk, :n], cb, S)
            V_hat = dequant(v_codes[b, hk, :n], v_radii[b, hk, :n], cb, S)
            for j in range(n_q):
                visible = n - (n_q - 1 - j)
                if visible <= 0:
                    continue
                for h in range(hk * group, (hk + 1) * group):
                    out[b, j, h] = softmax_attention(q[b, j, h], K_hat[:visible], V_hat[:visible], scale)
    return out


def log_sum_exp_scores(q: np.ndarray, K: np.ndarray, scale: float) -> float:
    """log of the softmax denominator of Eq. 2 for one query over the rows of K (-inf for no rows)."""
    if K.shape[0] == 0:
        return -np.inf
    s = (K @ q) * scale
    m = s.max()
    return float(m + np.log(np.sum(np.exp(s - m))))


def merge_attention(outs, lses):
    """Attention over a union of disjoint token sets from the attentions over the sets: with
    lse_p = log sum_{t in set p} exp(s_t), softmax over the union gives sum_p exp(lse_p - lse) out_p,
    lse = log sum_p exp(lse_p) (Eq. 2 with its sum split by set).  outs [P, ..., d], lses [P, ...].
    Returns (out, lse); rows whose sets are all empty give zeros and -inf."""
    outs = np.asarray(outs, dtype=np.float64)
    lses = np.asarray(lses, dtype=np.float64)
    top = lses.max(axis=0)
    safe = np.where(np.isfinite(top), top, 0.0)
    w = np.where(np.isfinite(lses), np.exp(lses - safe), 0.0)
    tot = w.sum(axis=0)
    out = np.sum(w[..., None] * np.where(np.isfinite(lses)[..., None], outs, 0.0), axis=0) / np.where(tot > 0, tot, 1.0)[..., None]
    with np.errstate(divide="ignore"):
        lse = np.where(tot > 0, safe + np.log(np.where(tot > 0, tot, 1.0)), -np.inf)
    return out, lse


def attention_with_tail(q, k_codes, k_radii, v_codes, v_radii, lens, cb: Codebooks, S, scale, k_tail, v_tail, tail_lens):
    """Eq. 2 over a cache whose first lens[b] tokens are PolarQuant-compressed and whose last tail_lens[b] tokens are
    kept as they are (the protocol of Section 5.3 for generated tokens): softmax over the dequantised keys followed
    by the exact tail keys, values likewise.  k_tail, v_tail [B, T, Hkv, d].  Returns (out [B, Hq, d], lse [B, Hq])."""
    q = np.asarray(q, dtype=np.float64)
    B, Hq, d = q.shape
    Hkv = k_codes.shape[1]
    group = Hq // Hkv
    out = np.zeros((B, Hq, d))
    lse = np.full((B, Hq), -np.inf)
    for b in range(B):
        n, t = int(lens[b]), int(tail_lens[b])
        for hk in range(Hkv):
            K = np.concatenate([dequant(k_codes[b, hk, :n], k_radii[b, hk, :n], cb, S), np.asarray(k_tail[b, :t, hk], dtype=np.float64)])
            V = np.concatenate([dequant(v_codes[b, hk, :n], v_radii[b, hk, :n], cb, S), np.asarray(v_tail[b, :t, hk], dtype=np.float64)])
            for h in range(hk * group, (hk + 1) * group):
                if n + t > 0:
                    out[b, h] = softmax_attention(q[b, h], K, V, scale)
                    lse[b, h] = log_sum_exp_scores(q[b, h], K, scale)
    return out, lse


def exact_attention(q, K, V, lens, scale):
    """Eq. 2 on the unquantised cache (quality information only, never a parity target).
    K, V: [B, Hkv, capacity, d]."""
    q = np.asarray(q, dtype=np.float64)
    B, Hq, d = q.shape
    Hkv = K.shape[1]
    group = Hq // Hkv
    out = np.zeros((B, Hq, d), dtype=np.float64)
    for b in range(B):
        n = int(lens[b])
        for h in range(Hq):
            hk = h // group
            out[b, h] = softmax_attention(q[b, h], np.asarray(K[b, hk, :n], dtype=np.float64),
                                          np.asarray(V[b, hk, :n], dtype=np.float64), scale)
    return out


# --------------------------------------------------------------------------------------
# A cache that grows (the stream of Section 4: encode a prefill chunk, append one token)
# --------------------------------------------------------------------------------------
class OracleCache:
    """Codes and radii of K and V for B sequences x Hkv heads with per-sequence lengths."""

    def __init__(self, batch: int, n_kv_heads: int, capacity: int, d: int, cb: Codebooks, S):
        self.cb, self.S, self.d = cb, np.asarray(S, dtype=np.float64), d
        n_codes = sum(d >> l for l in range(1, cb.n_levels + 1))
        n_radii = d >> cb.n_levels
        shape = (batch, n_kv_heads, capacity)
        self.k_codes = np.zeros(shape + (n_codes,), dtype=np.uint8)
        self.v_codes = np.zeros(shape + (n_codes,), dtype=np.uint8)
        self.k_radii = np.zeros(shape + (n_radii,), dtype=np.float16)
        self.v_radii = np.zeros(shape + (n_radii,), dtype=np.float16)
        self.lens = np.zeros(batch, dtype=np.int64)

    def encode_chunk(self, b: int, K: np.ndarray, V: np.ndarray):
        """Append a chunk of ``n`` tokens to sequence ``b``; K, V are [n, Hkv, d]."""
        n = K.shape[0]
        pos = int(self.lens[b])
        for hk in range(K.shape[1]):
            c, r, _ = encode(K[:, hk], self.S, self.cb)
            self.k_codes[b, hk, pos:pos + n], self.k_radii[b, hk, pos:pos + n] = c, r
            c, r, _ = encode(V[:, hk], self.S, self.cb)
            self.v_codes[b, hk, pos:pos + n], self.v_radii[b, hk, pos:pos + n] = c, r
        self.lens[b] = pos + n

    def append(self, k_new: np.ndarray, v_new: np.ndarray):
        """One new token for every sequence; k_new, v_new are [B, Hkv, d]."""
        for b in range(k_new.shape[0]):
            self.encode_chunk(b, k_new[b][None], v_new[b][None])

    def attend(self, q: np.ndarray, scale: float) -> np.ndarray:
        return decode_attention(q, self.k_codes, self.k_radii, self.v_codes, self.v_radii,
                                self.lens, self.cb, self.S, scale)


# --------------------------------------------------------------------------------------
# Accounting helpers used by the parity tests (not part of the method)
# --------------------------------------------------------------------------------------
def boundary_distance(angles, cb: Codebooks):
    """For every angle, the distance to the nearest decision point of its level: the
    interior boundaries, plus the wrap point 0 == 2*pi at level 1.  Same layout as the
    canonical code vector."""
    out = []
    for l, psi in enumerate(angles):
        pts = cb.boundaries[l]
        if l == 0:
            pts = np.concatenate(([0.0], pts, [TWO_PI]))
        out.append(np.min(np.abs(psi[..., None] - pts), axis=-1))
    return np.concatenate(out, axis=-1)
