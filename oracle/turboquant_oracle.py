"""Plain CPU oracle for TurboQuant (arxiv 2504.19874).

THIS IS TEST INFRASTRUCTURE, not a product path: a slow, literal, fp64 numpy
implementation of what the paper's Algorithm 1 (TurboQuant_mse) and
Algorithm 2 (TurboQuant_prod) compute, used only to check the CUDA library.
It shares no code, table or constant with the CUDA path and must never be
imported by it.  Only the tests, the smoke check and the benchmark's
cpu-baseline leg may call it.

Every function follows the paper's steps in the paper's order and notation;
no step is fused, folded or reordered (in particular the three d x d products
of Algorithm 2 are all taken, and scores are formed in the original basis from
the dequantised vectors).  Matrix products, QR, argmin and sort are library
primitives used as single steps.

Pins (see tests/test_oracle_pins.py): closed-form b=1 centroid, the large-d
centroids the paper prints for b=1,2, the distortion values of Theorems 1
and 2 and both pairs of bounds, Pi Pi^T = I, brute-force argmin on tiny d,
Monte-Carlo unbiasedness of the prod estimator, the 2/pi bias of the mse
estimator at b=1, the index entropy at b=4; the entropy coder of the indices:
dyadic probabilities, the worked example of RFC 1951 3.2.2, Kraft equality,
optimality against brute force, a hand-computed row stream, round trips.
`attend` (softmax-weighted sum over dequantised values) has no value in the
paper to pin against beyond its textbook softmax definition: parity unpinned.
`select_outlier_channels` is a harness rule the paper does not define:
parity unpinned.
"""
from __future__ import annotations

import math

import numpy as np
from scipy import special as _sp

_U64 = (1 << 64) - 1


# --------------------------------------------------------------------------
# Seeded Gaussian draws (counter-based, so both sides of a test can produce
# the same matrix from (seed, position) without sharing code).
# --------------------------------------------------------------------------
def _mix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on uint64 arrays (wrap-around arithmetic)."""
    x = x.copy()
    x ^= x >> np.uint64(30)
    x *= np.uint64(0xBF58476D1CE4E5B9)
    x ^= x >> np.uint64(27)
    x *= np.uint64(0x94D049BB133111EB)
    x ^= x >> np.uint64(31)
    return x


def counter_u64(seed: int, counters: np.ndarray) -> np.ndarray:
    """h(seed, ctr) = mix(mix(seed + G) + ctr * G), G = 0x9E3779B97F4A7C15."""
    g = np.uint64(0x9E3779B97F4A7C15)
    with np.errstate(over="ignore"):
        s = _mix64(np.array([(seed + 0x9E3779B97F4A7C15) & _U64], dtype=np.uint64))[0]
        return _mix64(s + counters.astype(np.uint64) * g)


def gaussian_matrix(rows: int, cols: int, seed: int) -> np.ndarray:
    """i.i.d. N(0,1) entries; element e = r*cols + c uses counters 2e, 2e+1
    through Box-Muller: sqrt(-2 ln u1) cos(2 pi u2),
    u1 = ((h>>11) + 0.5) 2^-53 in (0,1), u2 = (h>>11) 2^-53 in [0,1)."""
    e = np.arange(rows * cols, dtype=np.uint64)
    h1 = counter_u64(seed, e * np.uint64(2))
    h2 = counter_u64(seed, e * np.uint64(2) + np.uint64(1))
    u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 0.5) * 2.0 ** -53
    u2 = (h2 >> np.uint64(11)).astype(np.float64) * 2.0 ** -53
    g = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return g.reshape(rows, cols)


def rotation(d: int, seed: int) -> np.ndarray:
    """Random rotation Pi (Section 3.1): QR of a Gaussian matrix, made unique
    by taking Q diag(sign(diag R)) (the paper leaves the sign free)."""
    q, r = np.linalg.qr(gaussian_matrix(d, d, seed))
    sgn = np.where(np.diag(r) < 0.0, -1.0, 1.0)
    return q * sgn[None, :]


def projection(d: int, seed: int) -> np.ndarray:
    """QJL matrix S with i.i.d. N(0,1) entries (Definition 1, Algorithm 2)."""
    return gaussian_matrix(d, d, seed)


# --------------------------------------------------------------------------
# Lemma 1 density and the Lloyd-Max codebook of Eq. (4)
# --------------------------------------------------------------------------
def _log_density_constant(d: int) -> float:
    return math.lgamma(d / 2.0) - math.lgamma((d - 1) / 2.0) - 0.5 * math.log(math.pi)


def coordinate_density(x, d: int):
    """f_X(x) = Gamma(d/2) / (sqrt(pi) Gamma((d-1)/2)) (1 - x^2)^((d-3)/2), Lemma 1."""
    x = np.asarray(x, dtype=np.float64)
    return np.exp(_log_density_constant(d)) * np.power(1.0 - x * x, (d - 3) / 2.0)


def coordinate_cdf(x, d: int):
    """P[X <= x]: (1+X)/2 ~ Beta((d-1)/2, (d-1)/2) for the density of Lemma 1."""
    x = np.asarray(x, dtype=np.float64)
    a = (d - 1) / 2.0
    return _sp.betainc(a, a, (1.0 + x) / 2.0)


def _partial_first_moment(x, d: int):
    """Antiderivative of x f_X(x): -K (1 - x^2)^((d-1)/2) / (d - 1)."""
    x = np.asarray(x, dtype=np.float64)
    return -np.exp(_log_density_constant(d)) * np.power(1.0 - x * x, (d - 1) / 2.0) / (d - 1)


def codebook(d: int, b: int, tol: float = 1e-13, max_iter: int = 200000) -> np.ndarray:
    """2^b centroids c_1 <= ... <= c_{2^b} minimising Eq. (4) for f_X (Lloyd-Max).

    Alternates the two optimality conditions the paper states: boundaries are
    midpoints of consecutive centroids, and each centroid is the conditional
    mean of f_X on its cell.  Starts from the medians of 2^b equal-probability
    cells.  b = 0 gives the single centroid 0.
    """
    if d < 2:
        raise ValueError("d must be >= 2")
    k = 1 << b
    if k == 1:
        return np.zeros(1)
    a = (d - 1) / 2.0
    c = 2.0 * _sp.betaincinv(a, a, (np.arange(k) + 0.5) / k) - 1.0
    for _ in range(max_iter):
        t = np.concatenate(([-1.0], 0.5 * (c[:-1] + c[1:]), [1.0]))
        mass = np.diff(coordinate_cdf(t, d))
        first = np.diff(_partial_first_moment(t, d))
        new_c = first / mass
        new_c = 0.5 * (new_c - new_c[::-1])  # f_X is even: c_i = -c_{k+1-i}
        delta = np.max(np.abs(new_c - c))
        c = new_c
        if delta < tol:
            break
    else:
        raise RuntimeError("Lloyd-Max did not converge")
    return c


def index_probabilities(d: int, centroids: np.ndarray) -> np.ndarray:
    """p_l = integral of f_X over cell l (entropy-coding paragraph, Section 3.1)."""
    c = np.asarray(centroids, dtype=np.float64)
    t = np.concatenate(([-1.0], 0.5 * (c[:-1] + c[1:]), [1.0]))
    return np.diff(coordinate_cdf(t, d))


# --------------------------------------------------------------------------
# Bit packing (the paper only says "b-bit integers"; the layout is ours):
# coordinate j occupies bits [j*bits, (j+1)*bits) of the row's little-endian
# bit stream; bit p of the row is bit (p & 7) of byte (p >> 3); pad bits are 0.
# --------------------------------------------------------------------------
def pack_bits(values: np.ndarray, bits: int, row_bytes: int) -> np.ndarray:
    values = np.asarray(values)
    n, d = values.shape
    out = np.zeros((n, row_bytes), dtype=np.uint8)
    for j in range(d):
        for q in range(bits):
            p = j * bits + q
            out[:, p >> 3] |= (((values[:, j] >> q) & 1) << (p & 7)).astype(np.uint8)
    return out


def unpack_bits(packed: np.ndarray, bits: int, d: int) -> np.ndarray:
    packed = np.asarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    out = np.zeros((n, d), dtype=np.uint8)
    for j in range(d):
        for q in range(bits):
            p = j * bits + q
            out[:, j] |= (((packed[:, p >> 3] >> (p & 7)) & 1) << q).astype(np.uint8)
    return out


# --------------------------------------------------------------------------
# Algorithm 1: TurboQuant_mse
# --------------------------------------------------------------------------
def _unit(X: np.ndarray):
    """nu = ||x||, u = x / nu (Section 1.3: norms are stored separately and the
    unit vector is quantised).  A zero vector gives nu = 0 and u = 0."""
    X = np.asarray(X, dtype=np.float64)
    nu = np.sqrt(np.sum(X * X, axis=1))
    safe = np.where(nu > 0.0, nu, 1.0)
    return X / safe[:, None], nu


def rotate(U: np.ndarray, Pi: np.ndarray) -> np.ndarray:
    """y = Pi . x for every row x of U (Algorithm 1, Quant step 1)."""
    return np.asarray(U, dtype=np.float64) @ np.asarray(Pi, dtype=np.float64).T


def nearest_centroid(Y: np.ndarray, centroids: np.ndarray, chunk: int = 4096) -> np.ndarray:
    """idx_j = argmin_k |y_j - c_k| (Algorithm 1, Quant step 2); ties -> lower k."""
    c = np.asarray(centroids, dtype=np.float64)
    Y = np.asarray(Y, dtype=np.float64)
    idx = np.empty(Y.shape, dtype=np.uint8)
    for s in range(0, Y.shape[0], chunk):
        blk = Y[s:s + chunk]
        idx[s:s + chunk] = np.argmin(np.abs(blk[:, :, None] - c[None, None, :]), axis=2)
    return idx


def quant_mse(X, Pi, centroids):
    """Quant_mse: returns (idx [n,d] uint8, nu [n])."""
    U, nu = _unit(X)
    Y = rotate(U, Pi)
    return nearest_centroid(Y, centroids), nu


def dequant_mse_unit(idx, Pi, centroids):
    """DeQuant_mse: y~_j = c[idx_j]; x~ = Pi^T . y~ (unit-vector scale)."""
    c = np.asarray(centroids, dtype=np.float64)
    Yt = c[np.asarray(idx, dtype=np.int64)]
    return Yt @ np.asarray(Pi, dtype=np.float64)          # rows: (Pi^T y~)^T = y~^T Pi


def dequant_mse(idx, nu, Pi, centroids):
    """DeQuant_mse rescaled by the stored norm (Section 1.3)."""
    return dequant_mse_unit(idx, Pi, centroids) * np.asarray(nu, dtype=np.float64)[:, None]


# --------------------------------------------------------------------------
# Definition 1 (QJL) and Algorithm 2: TurboQuant_prod
# --------------------------------------------------------------------------
def qjl_quant(R, S):
    """Q_qjl(r) = sign(S . r) in {-1,+1}; sign(0) is taken as +1."""
    P = np.asarray(R, dtype=np.float64) @ np.asarray(S, dtype=np.float64).T
    return np.where(P >= 0.0, 1, -1).astype(np.int8), P


def qjl_dequant(Z, S):
    """Q_qjl^{-1}(z) = sqrt(pi/2) / d . S^T . z."""
    S = np.asarray(S, dtype=np.float64)
    d = S.shape[1]
    return math.sqrt(math.pi / 2.0) / d * (np.asarray(Z, dtype=np.float64) @ S)


def qjl_given_idx(X, idx, Pi, S, centroids):
    """Steps 2-4 of Quant_prod for a GIVEN idx: r = u - DeQuant_mse(idx),
    qjl = sign(S r), gamma = ||r||.  Returns (qjl, gamma, S r)."""
    U, nu = _unit(X)
    R = U - dequant_mse_unit(idx, Pi, centroids)
    R[nu == 0.0] = 0.0
    Z, P = qjl_quant(R, S)
    gamma = np.sqrt(np.sum(R * R, axis=1))
    return Z, gamma, P


def quant_prod(X, Pi, S, centroids):
    """Quant_prod with an MSE stage whose codebook is `centroids` (b-1 bits):
    returns (idx, qjl in {-1,+1}, gamma = ||r||, nu = ||x||)."""
    idx, nu = quant_mse(X, Pi, centroids)
    Z, gamma, _ = qjl_given_idx(X, idx, Pi, S, centroids)
    return idx, Z, gamma, nu


def dequant_prod(idx, qjl, gamma, nu, Pi, S, centroids):
    """DeQuant_prod: x~_mse + sqrt(pi/2)/d . gamma . S^T . qjl, times nu."""
    x_mse = dequant_mse_unit(idx, Pi, centroids)
    x_qjl = qjl_dequant(qjl, S) * np.asarray(gamma, dtype=np.float64)[:, None]
    return (x_mse + x_qjl) * np.asarray(nu, dtype=np.float64)[:, None]


# --------------------------------------------------------------------------
# Inner-product estimates, top-k, attention tail
# --------------------------------------------------------------------------
def score(Q, Xhat):
    """<q, x~> for every query row q and every dequantised vector x~
    (the estimator of Section 3.2 is the inner product with DeQuant's output)."""
    return np.asarray(Q, dtype=np.float64) @ np.asarray(Xhat, dtype=np.float64).T


def topk(scores, k: int):
    """k largest entries of each row, descending; equal scores -> lower id first."""
    scores = np.asarray(scores, dtype=np.float64)
    n = scores.shape[1]
    ids = np.empty((scores.shape[0], k), dtype=np.int64)
    for i, row in enumerate(scores):
        order = np.lexsort((np.arange(n), -row))
        ids[i] = order[:k]
    return np.take_along_axis(scores, ids, axis=1), ids


def attend(scores, Vhat, scale: float):
    """softmax(scale . scores) . V~  (decoder attention over a compressed cache)."""
    s = np.asarray(scores, dtype=np.float64) * scale
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ np.asarray(Vhat, dtype=np.float64)


def select_outlier_channels(X, count: int) -> np.ndarray:
    """Channels with the largest sum of squares over tokens (ties -> lower
    channel), ascending.  The paper defers this choice to prior work."""
    X = np.asarray(X, dtype=np.float64)
    energy = np.sum(X * X, axis=0)
    order = np.lexsort((np.arange(energy.size), -energy))
    return np.sort(order[:count])


# --------------------------------------------------------------------------
# Entropy coding of the indices (Section 3.1, "entropy encoding codebook
# pointers"): the index of a coordinate takes value l with probability p_l (the
# mass of the l-th cell), so a lossless prefix code brings the average bit width
# from b down towards the entropy of {p_l} (about 3.8 bits at b = 4).  The
# paper names no particular code; this is a Huffman code over the 2^b values
# (optimal among prefix codes), written out as the textbook algorithm, with the
# code words assigned canonically from the lengths as in RFC 1951, 3.2.2.
# Row format (the library's, stated in its header): every vector is coded on
# its own; bit p of the row stream is bit (p & 7) of byte (p >> 3), code words
# follow one another without gaps, each written from its most significant bit.
# --------------------------------------------------------------------------
def huffman_lengths(p) -> np.ndarray:
    """Code length per symbol of a Huffman code for probabilities p (all > 0): repeatedly merge the two least
    probable nodes; among equally probable nodes the one created earlier (leaves in symbol order first) goes first."""
    p = [float(v) for v in p]
    n = len(p)
    if n == 1:
        return np.array([0], dtype=np.uint8)
    nodes = [(p[s], s, (s,)) for s in range(n)]           # (probability, creation order, symbols below)
    depth = [0] * n
    created = n
    while len(nodes) > 1:
        nodes.sort(key=lambda t: (t[0], t[1]))
        a, b = nodes[0], nodes[1]
        for s in a[2] + b[2]:
            depth[s] += 1
        nodes = nodes[2:] + [(a[0] + b[0], created, a[2] + b[2])]
        created += 1
    return np.array(depth, dtype=np.uint8)


def canonical_codes(lengths) -> np.ndarray:
    """Code word (as an integer, most significant bit first) per symbol from the lengths: symbols sorted by
    (length, symbol) receive consecutive values, shifted left whenever the length grows (RFC 1951, 3.2.2)."""
    lengths = [int(v) for v in lengths]
    codes = [0] * len(lengths)
    code, prev = 0, 0
    for length, s in sorted((l, s) for s, l in enumerate(lengths) if l > 0):
        code <<= length - prev
        codes[s] = code
        code += 1
        prev = length
    return np.array(codes, dtype=np.uint32)


def entropy_encode_row(symbols, lengths, codes):
    """(bytes, number of bits) of one row's code stream."""
    bits = []
    for s in symbols:
        l, c = int(lengths[s]), int(codes[s])
        bits.extend((c >> (l - 1 - i)) & 1 for i in range(l))
    out = np.zeros((len(bits) + 7) // 8, dtype=np.uint8)
    for pos, b in enumerate(bits):
        out[pos >> 3] |= b << (pos & 7)
    return out, len(bits)


def entropy_decode_row(stream, count, lengths, codes) -> np.ndarray:
    """`count` symbols read back from a row stream, one bit at a time (prefix property)."""
    table = {(int(lengths[s]), int(codes[s])): s for s in range(len(lengths))}
    out = np.zeros(count, dtype=np.uint8)
    pos = 0
    for j in range(count):
        l, c = 0, 0
        while (l, c) not in table:
            c = (c << 1) | ((int(stream[pos >> 3]) >> (pos & 7)) & 1)
            l += 1
            pos += 1
        out[j] = table[(l, c)]
    return out
